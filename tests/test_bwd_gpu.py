"""Parity of bigbird_attn_bwd (CUDA-core gradient kernels) with the fp64 oracle's gradients, through the C-ABI.

Tolerances (max-abs): 1e-4 for fp32 tensors (fp32 arithmetic, sums over up to a few hundred rows); 3e-2 for bf16 tensors
(the gradients are rounded to bf16 on output; |dq|, |dk|, |dv| reach a few units)."""
import numpy as np
import pytest
import torch

import paper_2007_14062_b200 as bb
from paper_2007_14062_b200 import synth
from oracle import bigbird_oracle as O

pytestmark = pytest.mark.gpu
TOL = {"fp32": 1e-4, "bf16": 3e-2}


def _case(dtype, B, H, nb, lengths="full", mode=0, g=2, r=3, w=3, seed=7, b=64, D=64):
    return synth.Workload(f"bwd_{dtype}_{nb}", dtype, B, H, nb * b, D, b, w, g, r, mode, seed=seed, lengths=lengths)


CASES = [
    synth.WORKLOADS["c1_tiny_itc_fp32"],
    _case("fp32", 2, 2, 10, lengths="ragged:64:640"),
    _case("fp32", 1, 2, 7, mode=1, g=1, r=2),
    _case("fp32", 1, 2, 9, b=16, D=32, w=5),                    # another block size and head dimension
    _case("bf16", 2, 2, 12, lengths="ragged:100:768"),
    _case("bf16", 1, 2, 9, mode=1, r=0),
    _case("fp32", 1, 2, 8, b=84, mode=1, g=3, r=0),             # the paper's ETC block size (App. E tables)
    _case("fp32", 1, 2, 6, D=128),                              # the largest head dimension of the CUDA-core kernels
]


@pytest.mark.parametrize("wl", CASES, ids=lambda w: f"{w.name}_{w.lengths}_{w.mode}_{w.b}")
def test_gradients_match_the_oracle(wl):
    dev = torch.device("cuda:0")
    q, k, v = synth.make_qkv(wl)
    gen = torch.Generator().manual_seed(wl.seed + 100)
    dout = torch.randn(q.shape, generator=gen, dtype=torch.float32).to(q.dtype)
    kpm = synth.key_padding_mask(wl)
    if kpm is not None and wl.B > 1:
        kpm[1, 197:] = 0            # a length that is not a multiple of the block size
        kpm[1, :197] = 1
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    qd, kd, vd, dod = (t.to(dev) for t in (q, k, v, dout))
    md = None if kpm is None else kpm.to(dev)
    out = torch.empty_like(qd)
    lse = torch.empty(q.shape[:3], device=dev, dtype=torch.float32)
    bb.bigbird_attn_fwd_simt(qd, kd, vd, L, md, out, lse, wl.scale)
    dq, dk, dv = (torch.full_like(qd, float("nan")) for _ in range(3))
    bb.bigbird_attn_bwd(qd, kd, vd, out, lse, dod, L, md, dq, dk, dv, wl.scale)
    torch.cuda.synchronize()
    assert bb.bigbird_last_launch_count() == 2
    got = [t.float().cpu().numpy() for t in (dq, dk, dv)]
    assert all(np.isfinite(g).all() for g in got)
    gr = O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    want = O.attention_bwd(q.float().numpy(), k.float().numpy(), v.float().numpy(), dout.float().numpy(), gr,
                           None if kpm is None else kpm.numpy(), wl.scale)
    worst = 0.0
    for (bi, h), grads in want.items():
        for g_, w_ in zip(got, grads):
            worst = max(worst, float(np.abs(g_[bi, h] - w_).max()))
    assert worst <= TOL[wl.dtype], (wl.name, worst)
    if kpm is not None:                                         # padded rows: exactly zero
        pad = kpm.numpy() == 0
        for g_ in got:
            assert (g_.transpose(0, 2, 1, 3)[pad] == 0).all()
    L.close()


def test_bad_arguments_are_refused_without_a_launch():
    L = bb.bigbird_build_layout(512, 64, 3, 2, 3, 0, 2, 0)
    t = torch.empty(16, device="cuda:0", dtype=torch.float32)
    ptr = t.data_ptr()
    args = lambda **kw: [kw.get("q", ptr), ptr, ptr, ptr, kw.get("lse", ptr), ptr, L.handle, None, ptr, ptr, ptr, 1, 2, kw.get("N", 512),
                         kw.get("D", 64), 64, 0.125, 0, None]
    # (every call below fails its argument checks before anything is enqueued; a well-formed call is what the parity
    # test above makes)
    assert bb.lib().bigbird_attn_bwd(*args(q=None)) == -1
    assert bb.lib().bigbird_attn_bwd(*args(lse=None)) == -1
    assert bb.lib().bigbird_attn_bwd(*args(N=1024)) == -1       # layout built for another N
    assert bb.lib().bigbird_attn_bwd(*args(D=48)) == -2
    L.close()
