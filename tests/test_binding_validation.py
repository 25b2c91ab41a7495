"""The Python binding refuses tensors that would make a kernel read or write out of bounds (wrong size, dtype, device,
layout) with a ValueError, before the C call.  Runs without a GPU: stand-in tensor objects carry only the attributes
the checks read, and their data_ptr() fails the test if a check lets them through to the call."""
from __future__ import annotations

import pytest
import torch

import paper_2512_09196_b200 as tf


class Fake:
    is_cuda = True

    def __init__(self, shape, dtype=torch.bfloat16, device="cuda:0", contiguous=True):
        self.shape, self.dtype, self.device, self._c = tuple(shape), dtype, device, contiguous

    def dim(self):
        return len(self.shape)

    def is_contiguous(self):
        return self._c

    def numel(self):
        n = 1
        for s in self.shape:
            n *= s
        return n

    def data_ptr(self):
        raise AssertionError("an invalid tensor reached the C call")


R, C = 6, 64
X = Fake((R, C))
BAD_FULL = [Fake((R, C - 8)), Fake((R - 1, C)), Fake((R, C), torch.float32), Fake((R, C), device="cuda:1"),
            Fake((R, C), contiguous=False), Fake((R * C,))]
BAD_PARAM = [Fake((C - 1,)), Fake((C,), torch.float32), Fake((C,), device="cuda:1"), Fake((1, C)), Fake((C,), contiguous=False)]
BAD_STAT = [Fake((R - 1,), torch.float32), Fake((R,), torch.bfloat16), Fake((R,), torch.float32, device="cuda:1")]
G, ST = Fake((C,)), Fake((R,), torch.float32)


@pytest.mark.parametrize("bad", BAD_FULL)
def test_outputs_and_second_inputs_must_match_x(bad):
    for call in (lambda: tf.tf_softmax_fwd(X, bad), lambda: tf.tf_log_softmax_fwd(X, bad), lambda: tf.tf_softmax_fwd_noalloc(X, bad),
                 lambda: tf.tf_layernorm_fwd(X, G, G, 1e-5, y=bad), lambda: tf.tf_rmsnorm_fwd(X, G, 1e-6, y=bad),
                 lambda: tf.tf_softmax_bwd(X, bad), lambda: tf.tf_softmax_bwd(X, X, bad), lambda: tf.tf_log_softmax_bwd(X, bad),
                 lambda: tf.tf_add_rmsnorm_fwd(X, bad, G, 1e-6, h=X, y=X), lambda: tf.tf_add_rmsnorm_fwd(X, X, G, 1e-6, h=bad, y=X),
                 lambda: tf.tf_add_layernorm_fwd(X, X, G, G, 1e-5, h=X, y=bad), lambda: tf.tf_layernorm_bwd(X, G, bad, ST, ST),
                 lambda: tf.tf_rmsnorm_bwd(X, G, X, ST, dx=bad), lambda: tf.tf_copy(X, bad)):
        with pytest.raises(ValueError):
            call()


@pytest.mark.parametrize("bad", BAD_PARAM)
def test_parameter_vectors_must_be_cols_long_and_of_x_dtype(bad):
    for call in (lambda: tf.tf_layernorm_fwd(X, bad, G, 1e-5, y=X), lambda: tf.tf_layernorm_fwd(X, G, bad, 1e-5, y=X),
                 lambda: tf.tf_rmsnorm_fwd(X, bad, 1e-6, y=X), lambda: tf.tf_add_layernorm_fwd(X, X, G, bad, 1e-5, h=X, y=X),
                 lambda: tf.tf_add_rmsnorm_fwd(X, X, bad, 1e-6, h=X, y=X), lambda: tf.tf_layernorm_bwd(X, bad, X, ST, ST),
                 lambda: tf.tf_rmsnorm_bwd(X, bad, X, ST), lambda: tf.tf_tune("layernorm", R, C, tf.TF_BF16, like=(X, bad, G))):
        with pytest.raises(ValueError):
            call()


@pytest.mark.parametrize("bad", BAD_STAT)
def test_row_statistics_must_be_fp32_rows_long(bad):
    for call in (lambda: tf.tf_layernorm_fwd(X, G, G, 1e-5, y=X, mean=bad, rstd=ST), lambda: tf.tf_layernorm_fwd(X, G, G, 1e-5, y=X, mean=ST, rstd=bad),
                 lambda: tf.tf_rmsnorm_fwd(X, G, 1e-6, y=X, rstd=bad), lambda: tf.tf_layernorm_bwd(X, G, X, bad, ST),
                 lambda: tf.tf_layernorm_bwd(X, G, X, ST, bad), lambda: tf.tf_rmsnorm_bwd(X, G, X, bad)):
        with pytest.raises(ValueError):
            call()


def test_cpu_tensors_and_unsupported_dtypes_are_refused():
    with pytest.raises(ValueError):
        tf.tf_softmax_fwd(torch.zeros(4, 8))
    with pytest.raises(ValueError):
        tf.tf_softmax_fwd(Fake((4, 8), contiguous=False), Fake((4, 8)))
    with pytest.raises(ValueError):
        tf.tf_tune("softmax", R, C + 8, tf.TF_BF16, like=(X, None, None))
