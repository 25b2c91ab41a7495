"""The library's calls inside a CUDA graph: every entry point only enqueues work on the caller's stream (no hidden
synchronisation, no allocation by the library itself), so a sequence of calls can be captured once and replayed on new
data -- the way to run launch-bound shapes.  The replay must give, bit for bit, what the same calls give eagerly on the
same inputs, and those are checked against the oracle."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu
BF16 = inputs.BF16


def _bits(t):
    return t.view(torch.uint16) if t.dtype == torch.bfloat16 else t.view(torch.int32)


def _block(x, r, gamma, beta, w, dy):
    """A residual update with both norms, a softmax over the result and the backward passes of the norms."""
    h, y, mean, rstd = tf.tf_add_layernorm_fwd(x, r, gamma, beta, 1e-5)
    h2, z, rr = tf.tf_add_rmsnorm_fwd(h, y, w, 1e-6, want_rstd=True)
    p = tf.tf_softmax_fwd(z)
    lp = tf.tf_log_softmax_fwd(z)
    dp = tf.tf_softmax_bwd(p, dy)
    dx, dgamma, dbeta = tf.tf_layernorm_bwd(h, gamma, dp, mean, rstd)
    dz, dw = tf.tf_rmsnorm_bwd(h2, w, dy, rr)
    return [h, y, mean, rstd, h2, z, rr, p, lp, dp, dx, dgamma, dbeta, dz, dw]


@pytest.mark.parametrize("rows,cols", [(64, 1024), (512, 4096)])
def test_a_captured_sequence_replays_on_new_data(rows, cols):
    def fresh(seed):
        mk = lambda s, mean, std: parity.to_dev(inputs.normal((rows, cols), BF16, seed, s, mean, std), BF16)
        return mk(0, 0.3, 2.0), mk(7, -0.2, 1.0), mk(3, 0.0, 1.0)
    gamma = parity.to_dev(inputs.uniform((cols,), BF16, 5, 1, 0.5, 1.5), BF16)
    beta = parity.to_dev(inputs.normal((cols,), BF16, 5, 2, 0.0, 0.1), BF16)
    w = parity.to_dev(inputs.normal((cols,), BF16, 5, 4, 1.0, 0.1), BF16)
    x, r, dy = fresh(11)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                                  # first use outside the capture (plans, status word, torch's pools)
        for _ in range(2):
            _block(x, r, gamma, beta, w, dy)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    launches_before = tf.tf_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        outs = _block(x, r, gamma, beta, w, dy)
    assert tf.tf_launch_count() > launches_before                  # the library's own kernels are what was captured
    for seed in (21, 22):
        nx, nr, ndy = fresh(seed)
        x.copy_(nx); r.copy_(nr); dy.copy_(ndy)
        graph.replay()
        torch.cuda.synchronize()
        tf.tf_device_status()
        replayed = [o.clone() for o in outs]
        eager = _block(nx, nr, gamma, beta, w, ndy)
        torch.cuda.synchronize()
        for i, (a, b) in enumerate(zip(replayed, eager)):
            assert torch.equal(_bits(a), _bits(b)), (rows, cols, seed, i)
    # and the eager results are the oracle's: the fused add + LayerNorm of the last inputs
    import oracle
    xh, rh = parity.to_host(nx, BF16), parity.to_host(nr, BF16)
    h_ref = oracle.add(xh, rh, BF16)
    np.testing.assert_array_equal(parity.to_host(replayed[0], BF16), h_ref)
    wl = inputs.Workload("graph-ln", "layernorm", BF16, rows, cols, seed=1, eps=1e-5)
    data = {"x": h_ref, "gamma": parity.to_host(gamma, BF16), "beta": parity.to_host(beta, BF16)}
    got = {"y": parity.to_host(replayed[1], BF16), "mean": replayed[2].cpu().numpy(), "rstd": replayed[3].cpu().numpy()}
    fails = parity.check(wl, data, got, parity.run_oracle(wl, data))
    assert not fails, fails
