"""The calibration kernels through the C ABI: the streaming copy is exact for every size and alignment, the
element-wise sine matches the CPU oracle for every launch geometry."""
from __future__ import annotations

import numpy as np
import pytest
import torch

import compare
import oracle
import paper_2512_09196_b200 as tf
from paper_2512_09196_b200 import inputs
import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("nbytes", [1, 15, 16, 17, 4096, 65537, (64 << 20) + 5])
def test_copy_is_exact(nbytes):
    src = torch.randint(0, 256, (nbytes + 64,), dtype=torch.uint8, device="cuda")
    for off_in, off_out in ((0, 0), (16, 32), (1, 0), (3, 5)):
        dst = torch.full((nbytes + 64,), 7, dtype=torch.uint8, device="cuda")
        st = tf.lib().tf_copy(src.data_ptr() + off_in, dst.data_ptr() + off_out, nbytes, torch.cuda.current_stream().cuda_stream)
        assert st == 0
        torch.cuda.synchronize()
        assert torch.equal(dst[off_out:off_out + nbytes], src[off_in:off_in + nbytes])
        assert (dst[:off_out] == 7).all() and (dst[off_out + nbytes:] == 7).all()       # nothing written outside


@pytest.mark.parametrize("dt", [inputs.F32, inputs.BF16])
def test_sin_matches_the_oracle_for_every_geometry(dt):
    for n, std in ((1, 1.0), (7, 1.0), (4099, 1.0), (1 << 20, 3.0), (100003, 1000.0), (100003, 2.0e4), (4099, 1.0e20)):
        x = inputs.normal((n,), dt, seed=n, stream=0, mean=0.0, std=std)
        ref, ref64 = oracle.sin(x, dt, want64=True)
        for threads, per_sm, offset in ((0, 0, 0), (32, 1, 0), (1024, 2, 0), (128, 8, 1)):
            xd = parity.to_dev(x, dt, offset)
            y = tf.tf_sin_fwd(xd, parity.guarded(tuple(xd.shape), xd.dtype, offset, name="y"), threads, per_sm)
            torch.cuda.synchronize()
            r = compare.compare_values(parity.to_host(y, dt), ref, ref64, dt)
            assert r.ok, (n, std, threads, per_sm, offset, str(r))
    L = tf.lib()
    p = torch.zeros(64, device="cuda").data_ptr()
    assert L.tf_sin_fwd(p, p, 8, 0, 48, 1, None) == 1            # threads not a multiple of 32
    assert L.tf_sin_fwd(p, p, 8, 0, 64, 3, None) == 1            # vectors per thread must be 1, 2, 4 or 8
    assert L.tf_sin_fwd(None, p, 8, 0, 0, 0, None) == 1
    assert L.tf_copy(None, p, 8, None) == 1 and L.tf_copy(p, p, 0, None) == 0
