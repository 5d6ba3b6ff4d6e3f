"""bigbird_attn_fwd_static: the forward pass for callers that must not allocate device memory.

Some users of the library run where a cudaMalloc is not an option: their GPU memory belongs to a pool that was
sized once at start-up, or they sit in a serving loop where the implicit synchronisation of an allocation is
too expensive.  For them the library has one entry point whose scratch is a fixed array inside the loaded
module.  This test calls it through the C ABI and checks that it returns what the ordinary entry point
returns -- and what the fp64 oracle says, so that a fault shared by both entry points cannot hide -- on two
calls in a row with different problems (the second must not see anything the first one left in the shared
array), and that a problem beyond the array's limits is refused.

The file name makes pytest collect it last, so a run that stops at the first failure has already run
everything else.  It does not depend on any other test having run.
"""
import numpy as np
import pytest
import torch

import paper_2007_14062_b200 as bb
from paper_2007_14062_b200 import synth
from oracle import bigbird_oracle as O

pytestmark = pytest.mark.gpu

TOL_OUT, TOL_LSE = 2e-2, 1e-3       # the bf16 tolerances of tests/test_parity_gpu.py


def _both(wl, kpm_edit=None):
    dev = torch.device("cuda:0")
    q, k, v = (t.to(dev) for t in synth.make_qkv(wl))
    kpm = synth.key_padding_mask(wl)
    if kpm is not None and kpm_edit is not None:
        kpm_edit(kpm)
    md = None if kpm is None else kpm.to(dev)
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    res = []
    for fn in (bb.bigbird_attn_fwd, bb.bigbird_attn_fwd_static):
        out = torch.full_like(q, float("nan"))
        lse = torch.full(q.shape[:3], float("nan"), device=dev, dtype=torch.float32)
        fn(q, k, v, L, md, out, lse, wl.scale)
        torch.cuda.synchronize()
        res.append((out.float().cpu().numpy(), lse.cpu().numpy()))
    st, detail = bb.bigbird_last_status()
    assert st == 0, (st, detail)
    assert bb.bigbird_last_status_static() == (0, 0)      # the static call's own status words, read without allocating
    L.close()
    # the static entry point against the oracle as well
    gr = O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    want = O.attention(q.float().cpu().numpy(), k.float().cpu().numpy(), v.float().cpu().numpy(), gr,
                       None if kpm is None else kpm.numpy(), wl.scale)
    o_new, l_new = res[1]
    for (bi, h), (wo, wlse) in want.items():
        vb = np.ones(wl.N, dtype=bool) if kpm is None else kpm[bi].numpy() != 0
        assert np.abs(o_new[bi, h][vb] - wo[vb]).max(initial=0) <= TOL_OUT, (wl.name, bi, h)
        assert np.abs(l_new[bi, h][vb] - wlse[vb]).max(initial=0) <= TOL_LSE, (wl.name, bi, h)
    return res, (None if kpm is None else kpm.numpy() != 0)


def _check(res, valid):
    (o_ref, l_ref), (o_new, l_new) = res
    assert not np.isnan(o_new).any() and not np.isnan(l_new).any()
    if valid is None:
        assert np.isfinite(l_new).all()
        assert np.abs(o_new - o_ref).max() <= TOL_OUT and np.abs(l_new - l_ref).max() <= TOL_LSE
        return
    for bi in range(o_ref.shape[0]):
        vb = valid[bi]
        assert np.abs(o_new[bi][:, vb] - o_ref[bi][:, vb]).max(initial=0) <= TOL_OUT
        assert np.abs(l_new[bi][:, vb] - l_ref[bi][:, vb]).max(initial=0) <= TOL_LSE
        assert (o_new[bi][:, ~vb] == 0).all() and np.isneginf(l_new[bi][:, ~vb]).all()     # padded query rows


def test_static_entry_point_matches_the_allocating_one_twice_in_a_row():
    # first call: several tiles per head, a ragged batch with a length that is not a multiple of the block size
    big = synth.Workload("noalloc_a", "bf16", 3, 4, 40 * 64, 64, 64, 3, 2, 3, 0, seed=11, lengths="ragged:300:2560")

    def edit(kpm):
        kpm[1, 1000:] = 0
        kpm[1, :1000] = 1

    res, valid = _both(big, edit)
    _check(res, valid)
    # second call, right after: a smaller problem with another layout (ETC, no random blocks) and no mask
    small = synth.Workload("noalloc_b", "bf16", 1, 2, 9 * 64, 64, 64, 3, 2, 0, 1, seed=12)
    res, valid = _both(small)
    _check(res, valid)


def test_static_entry_point_reuses_the_uploaded_schedule():
    """Two calls with one layout handle: the second sends no schedule (the array still holds it) and must give
    the same bits; a call with another handle in between replaces the schedule and the first handle's next
    call uploads again."""
    dev = torch.device("cuda:0")
    wl = synth.Workload("noalloc_c", "bf16", 2, 2, 12 * 64, 64, 64, 3, 2, 3, 0, seed=13)
    other = synth.Workload("noalloc_d", "bf16", 1, 2, 10 * 64, 64, 64, 3, 2, 1, 0, seed=14)
    q, k, v = (t.to(dev) for t in synth.make_qkv(wl))
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    outs = []
    for rep in range(3):
        out = torch.full_like(q, float("nan"))
        lse = torch.full(q.shape[:3], float("nan"), device=dev, dtype=torch.float32)
        bb.bigbird_attn_fwd_static(q, k, v, L, None, out, lse, wl.scale)
        torch.cuda.synchronize()
        outs.append((out.float().cpu().numpy(), lse.cpu().numpy()))
        if rep == 1:                                    # another layout takes the array over
            q2, k2, v2 = (t.to(dev) for t in synth.make_qkv(other))
            L2 = bb.bigbird_build_layout(other.N, other.b, other.w, other.g, other.r, other.seed, other.H, other.mode)
            bb.bigbird_attn_fwd_static(q2, k2, v2, L2, None, torch.empty_like(q2), None, other.scale)
            torch.cuda.synchronize()
            L2.close()
    assert bb.bigbird_last_status_static() == (0, 0)
    for o, l in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(l, outs[0][1])
    ref = torch.full_like(q, float("nan"))
    ref_lse = torch.full(q.shape[:3], float("nan"), device=dev, dtype=torch.float32)
    bb.bigbird_attn_fwd(q, k, v, L, None, ref, ref_lse, wl.scale)
    torch.cuda.synchronize()
    assert np.abs(ref.float().cpu().numpy() - outs[0][0]).max() <= TOL_OUT
    assert np.abs(ref_lse.cpu().numpy() - outs[0][1]).max() <= TOL_LSE
    L.close()


def test_static_entry_point_refuses_what_does_not_fit():
    # 131072 schedule steps is the limit of the fixed array; this layout needs more.  Nothing is launched.
    L = bb.bigbird_build_layout(1024 * 64, 64, 3, 2, 3, 0, 20, 0)
    _, _, _, steps = L.schedule()
    assert len(steps) > 131072
    fake = torch.empty(16, device="cuda:0", dtype=torch.bfloat16)
    code = bb.lib().bigbird_attn_fwd_static(fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), L.handle, None, fake.data_ptr(),
                                            None, 1, 20, 1024 * 64, 64, 64, 0.125, bb.BIGBIRD_BF16, None)
    assert code == -6 and "fixed scratch" in bb.bigbird_strerror(code)
    L.close()
    # fp32 tensors go to the CUDA-core kernel in bigbird_attn_fwd; the static entry point has no such path
    L = bb.bigbird_build_layout(512, 64, 3, 2, 3, 0, 2, 0)
    code = bb.lib().bigbird_attn_fwd_static(fake.data_ptr(), fake.data_ptr(), fake.data_ptr(), L.handle, None, fake.data_ptr(),
                                            None, 1, 2, 512, 64, 64, 0.125, bb.BIGBIRD_FP32, None)
    assert code == -2
    L.close()
