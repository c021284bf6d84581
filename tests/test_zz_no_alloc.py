"""The allocation-free salience entry point against the regular one and against the fp64 oracle.

`mvla_salience_noalloc` exists for callers that cannot allocate device memory when they call into
the library (frozen memory pools, real-time loops): its scratch is a fixed array in the library
image that every call on the device shares and that keeps the previous call's contents.  So the
check is made on two calls in a row with different problems: the second must not be disturbed by
what the first left behind.  This file is collected last on purpose."""
import numpy as np
import pytest
import torch

import oracle
from paper_2604_09244_b200 import mvla
from paper_2604_09244_b200 import workloads as W
from parity_util import SALIENCE_ATOL, SALIENCE_RTOL, device_tensors

pytestmark = pytest.mark.gpu


def _both(wl, check_no_allocation=False):
    dev = device_tensors(wl)
    ctx = mvla.context_for(wl)
    ref, _ = ctx.salience(wl.samples, dev["q"], dev["k"])
    out = torch.full((wl.total_vis,), -1.0, dtype=torch.float32, device="cuda")   # the caller's own buffer
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    stats0 = torch.cuda.memory_stats()["allocation.all.allocated"]
    mvla.salience_noalloc(wl.samples, dev["q"], dev["k"], out)
    torch.cuda.synchronize()
    if check_no_allocation:      # not on a device's first call: the driver loads the module then
        assert torch.cuda.mem_get_info()[0] == free0, "the call changed the free device memory"
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == stats0, "the call went through torch's allocator"
    ctx.close()
    return out, ref


def _oracle_scores(wl):
    t = wl.steps[0]
    return np.concatenate([oracle.salience(t.q, t.k, wl.n_heads, wl.head_dim, s) for s in wl.samples])


def _close_to_oracle(out, wl):
    ref = _oracle_scores(wl)
    got = out.cpu().numpy().astype(np.float64)
    return bool((np.abs(got - ref) <= SALIENCE_RTOL * np.abs(ref) + SALIENCE_ATOL).all())


def test_noalloc_matches_regular_entry_point_on_two_calls_in_a_row():
    first = W.small_workload(71, batch=3, D=256, H=4, d=128, dtype="bf16", n_txt=(5, 19, 33),
                             n_2d=(70, 130, 260), n_3d=(150, 37, 300))
    second = W.small_workload(72, batch=2, D=256, H=4, d=128, dtype="bf16", n_txt=(40, 7), n_2d=(33, 200),
                              n_3d=(90, 10))            # smaller: stale scratch entries lie beyond its range
    for n, wl in enumerate((first, second)):
        out, ref = _both(wl, check_no_allocation=n > 0)
        assert torch.isfinite(out).all()
        err = (out - ref).abs()
        assert bool((err <= SALIENCE_RTOL * ref.abs() + SALIENCE_ATOL).all())     # the regular entry point
        assert _close_to_oracle(out, wl)                                           # and the fp64 oracle itself
        assert abs(float(out[:wl.samples[0].n_vis].sum()) - 1.0) < 1e-4


def test_noalloc_fp32_and_capacity_limit():
    wl = W.config1_tiny()
    out, ref = _both(wl)
    assert bool(((out - ref).abs() <= SALIENCE_RTOL * ref.abs() + SALIENCE_ATOL).all())
    assert _close_to_oracle(out, wl)
    # 32 heads x 4097 visual tokens is past the fixed array: refused, nothing launched
    big = W.layout_2d_3d_txt(0, 8, 2049, 2047)
    big2 = W.layout_2d_3d_txt(big.seq_len, 8, 1, 0)
    q = torch.zeros(big.seq_len + big2.seq_len, 32, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(4097, dtype=torch.float32, device="cuda")
    with pytest.raises(mvla.MvlaError) as e:
        mvla.salience_noalloc([big, big2], q, q, out)
    assert e.value.code == mvla.ERR_CAPACITY
