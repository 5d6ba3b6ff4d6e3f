"""Parity of the CUDA library against the fp64 oracle, through the C-ABI (needs a B200).

Tolerances (max-abs): out 1e-5 for fp32 tensors, 2e-2 for bf16 tensors (fp32 accumulation); lse 1e-3.
Padded query rows are not compared with the oracle; the library's own contract for them (out = 0,
lse = -inf) is checked instead.
"""
import math

import numpy as np
import pytest
import torch

import paper_2007_14062_b200 as bb
from paper_2007_14062_b200 import synth
from oracle import bigbird_oracle as O

pytestmark = pytest.mark.gpu

TOL_OUT = {"fp32": 1e-5, "bf16": 2e-2}
TOL_LSE = 1e-3
IMPLS = {"fwd": bb.bigbird_attn_fwd, "simt": bb.bigbird_attn_fwd_simt}


def _graph(wl):
    return O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)


def _run(wl, q, k, v, kpm, impl="fwd", want_lse=True):
    dev = torch.device("cuda:0")
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    md = None if kpm is None else kpm.to(dev)
    out = torch.full_like(qd, float("nan"))
    lse = torch.full(q.shape[:3], float("nan"), device=dev, dtype=torch.float32) if want_lse else None
    IMPLS[impl](qd, kd, vd, L, md, out, lse, wl.scale)
    st, detail = bb.bigbird_last_status()
    assert st == 0, (st, detail)
    assert bb.bigbird_last_launch_count() >= 1
    res = out.float().cpu().numpy(), (None if lse is None else lse.cpu().numpy())
    L.close()
    return res


def _compare(wl, q, k, v, kpm, out, lse, slices, rows=None):
    gr = _graph(wl)
    qn, kn, vn = (t.float().numpy() for t in (q, k, v))      # the exact values handed to the GPU, widened
    kp = None if kpm is None else kpm.numpy()
    want = O.attention(qn, kn, vn, gr, kp, wl.scale, slices=slices, rows=rows)
    rws = np.arange(wl.N) if rows is None else np.asarray(rows)
    worst_o = worst_l = 0.0
    for (bi, h), (wo, wlse) in want.items():
        valid = np.ones(len(rws), dtype=bool) if kp is None else (kp[bi][rws] != 0)
        go, gl = out[bi, h][rws], lse[bi, h][rws]
        assert np.isfinite(go).all() and not np.isnan(gl).any()
        if valid.any():
            worst_o = max(worst_o, np.abs(go[valid] - wo[valid]).max())
            worst_l = max(worst_l, np.abs(gl[valid] - wlse[valid]).max())
        if (~valid).any():                                   # library contract for padded query rows
            assert (go[~valid] == 0).all() and np.isneginf(gl[~valid]).all()
    assert worst_o <= TOL_OUT[wl.dtype], (wl.name, worst_o)
    assert worst_l <= TOL_LSE, (wl.name, worst_l)
    return worst_o, worst_l


def _small(dtype, B, H, nb, lengths="full", mode=0, g=2, r=3, w=3, seed=7, sigma=1.0):
    return synth.Workload(f"small_{dtype}_{nb}", dtype, B, H, nb * 64, 64, 64, w, g, r, mode, seed=seed, sigma=sigma,
                          lengths=lengths)


# ------------------------------------------------------------------------------------------------ config 1
@pytest.mark.parametrize("impl", ["fwd", "simt"])
def test_c1_tiny_itc_fp32_every_element(impl):
    wl = synth.WORKLOADS["c1_tiny_itc_fp32"]
    q, k, v = synth.make_qkv(wl)
    out, lse = _run(wl, q, k, v, None, impl)
    _compare(wl, q, k, v, None, out, lse, slices=None)


# ------------------------------------------------------------------------------------------------ small, several tiles + ragged tails
SMALL = [
    _small("bf16", 2, 3, 11),                                   # odd block count: one unpaired tile
    _small("bf16", 2, 2, 12, lengths="ragged:100:768"),
    _small("bf16", 1, 2, 9, mode=1, r=0),                       # ETC
    _small("bf16", 1, 2, 16, g=3, r=2, w=5),
    _small("bf16", 1, 1, 4, g=4, r=0),                          # every block global
    _small("bf16", 1, 2, 6, g=0, r=1),                          # no global block
    _small("bf16", 1, 1, 1, g=1, r=0),                          # a single block
    _small("bf16", 1, 2, 131, lengths="fixed:7000"),            # long sequence: the global tile is split along the keys
    _small("bf16", 2, 1, 100, g=3, r=2),                        # split global tiles, an unpaired global block
    _small("bf16", 1, 1, 120, w=101, lengths="fixed:7000"),     # wide window: a sparse tile's key list spans two posted segments
    _small("fp32", 2, 2, 10, lengths="ragged:64:640"),
    _small("fp32", 1, 2, 7, mode=1, g=1, r=2),
]


@pytest.mark.parametrize("impl", ["fwd", "simt"])
@pytest.mark.parametrize("wl", SMALL, ids=lambda w: f"{w.name}_{w.lengths}_{w.mode}_{w.g}{w.r}{w.w}")
def test_small_cases_every_element(wl, impl):
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    if kpm is not None and wl.B > 1:
        kpm[1, 197:] = 0            # a length that is not a multiple of the block size
        kpm[1, :197] = 1
    out, lse = _run(wl, q, k, v, kpm, impl)
    _compare(wl, q, k, v, kpm, out, lse, slices=None)


# Head dimensions other than 64 exist on the CUDA-core path only (the tensor-core kernel is D = 64).
@pytest.mark.parametrize("dtype,D", [("fp32", 128), ("bf16", 128), ("fp32", 32)])
def test_other_head_dimensions_on_the_cuda_core_path(dtype, D):
    wl = synth.Workload(f"headdim_{dtype}_{D}", dtype, 2, 2, 9 * 64, D, 64, 3, 2, 3, 0, seed=31, lengths="ragged:100:576")
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    out, lse = _run(wl, q, k, v, kpm, "simt")
    _compare(wl, q, k, v, kpm, out, lse, slices=None)


# The paper's own ETC settings have block sizes that are not powers of two and global token counts that are not whole
# blocks (App. E hyper-parameter tables: ETC base, block 84, 230 global tokens, window 252 = 3 blocks; QA large, block
# 169, 430 global tokens, window 507 = 3 blocks; no random blocks).  The CUDA-core path takes any block size; the
# global tokens take the first g = 3 blocks and the unused tail of the third one is masked out as padding, which is the
# same graph for the tokens that exist.
PAPER_ETC = [
    ("etc_base_b84", synth.Workload("etc_b84", "fp32", 1, 2, 84 * (3 + 9), 64, 84, 3, 3, 0, 1, seed=21), 230),
    ("etc_base_b84_bf16", synth.Workload("etc_b84_bf16", "bf16", 2, 2, 84 * (3 + 7), 64, 84, 3, 3, 0, 1, seed=22), 230),
    ("qa_large_b169", synth.Workload("qa_b169", "fp32", 1, 2, 169 * (3 + 5), 64, 169, 3, 3, 0, 1, seed=23), 430),
]


@pytest.mark.parametrize("name,wl,g_tokens", PAPER_ETC, ids=[c[0] for c in PAPER_ETC])
def test_paper_etc_block_sizes_on_the_cuda_core_path(name, wl, g_tokens):
    q, k, v = synth.make_qkv(wl)
    kpm = torch.ones(wl.B, wl.N, dtype=torch.uint8)
    kpm[:, g_tokens:wl.g * wl.b] = 0                           # the global slots beyond the paper's count
    if wl.B > 1:
        kpm[1, wl.N - 100:] = 0                                # and a shorter sequence
    out, lse = _run(wl, q, k, v, kpm, "simt")
    _compare(wl, q, k, v, kpm, out, lse, slices=None)
    # the tensor-core entry point says so instead of computing something else
    if wl.dtype == "bf16":
        dev = torch.device("cuda:0")
        L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
        qd = q.to(dev)
        with pytest.raises(bb.BigBirdError) as ei:
            bb.bigbird_attn_fwd(qd, qd, qd, L, None, torch.empty_like(qd), None, wl.scale)
        assert ei.value.code == -2                              # BIGBIRD_EUNSUPPORTED
        L.close()


@pytest.mark.parametrize("impl", ["fwd", "simt"])
def test_fully_padded_sequence_and_no_lse(impl):
    wl = _small("bf16", 2, 2, 8)
    q, k, v = synth.make_qkv(wl)
    kpm = torch.ones((2, wl.N), dtype=torch.uint8)
    kpm[0] = 0                                                    # sequence 0 has no real token at all
    out, lse = _run(wl, q, k, v, kpm, impl)
    assert (out[0] == 0).all() and np.isneginf(lse[0]).all()
    _compare(wl, q, k, v, kpm, out, lse, slices=[(1, 0), (1, 1)])
    out2, none = _run(wl, q, k, v, kpm, impl, want_lse=False)
    assert none is None and np.array_equal(out, out2)


@pytest.mark.parametrize("impl", ["fwd", "simt"])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_closed_forms_on_gpu(impl, dtype):
    """V == 1 gives out == 1; Q == 0 gives lse = ln(#attended valid keys) and out = mean of attended V."""
    wl = _small(dtype, 1, 2, 12, lengths="fixed:700")
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    out, _ = _run(wl, q, k, torch.ones_like(v), kpm, impl)
    valid = kpm[0].numpy() != 0
    # (fp32: numerator and denominator are the same sum taken in two orders; a few dozen fp32 roundings apart)
    assert np.abs(out[0][:, valid] - 1).max() <= (4e-6 if dtype == "fp32" else 2 ** -8)
    out, lse = _run(wl, torch.zeros_like(q), k, v, kpm, impl)
    gr = _graph(wl)
    for h in range(wl.H):
        A = O.build_mask(gr, h) & valid[None, :]
        cnt = A.sum(axis=1)
        assert np.abs(lse[0, h][valid] - np.log(cnt[valid])).max() < 1e-4
        mean = (A.astype(np.float64) @ v[0, h].double().numpy()) / np.maximum(cnt, 1)[:, None]
        assert np.abs(out[0, h][valid] - mean[valid]).max() <= TOL_OUT[dtype]


def test_two_runs_are_bit_identical():
    wl = _small("bf16", 2, 4, 16, lengths="ragged:128:1024")
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    a = _run(wl, q, k, v, kpm)
    b = _run(wl, q, k, v, kpm)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])


def test_bounded_wait_expires_with_a_status_and_the_context_stays_usable():
    """A wait that nothing will ever satisfy gives up after its limit: the kernel returns, the status word says
    BIGBIRD_ETIMEOUT (-4) with the code of the wait, reading it clears it, and the next forward call is fine."""
    assert bb.bigbird_last_status() == (0, 0)
    bb.bigbird_selftest_wait_expiry()
    assert bb.bigbird_last_status() == (-4, 99)
    assert bb.bigbird_last_status() == (0, 0)
    wl = _small("bf16", 1, 2, 8)
    q, k, v = synth.make_qkv(wl)
    out, lse = _run(wl, q, k, v, None)
    _compare(wl, q, k, v, None, out, lse, slices=None)


# ------------------------------------------------------------------------------------------------ full-size workloads
def _sample_slices(wl, n, seed=0):
    rng = np.random.default_rng(seed)
    idx = rng.choice(wl.B * wl.H, size=min(n, wl.B * wl.H), replace=False)
    return sorted((int(i) // wl.H, int(i) % wl.H) for i in idx)


def test_c2_base_itc_bf16_full_size():
    wl = synth.WORKLOADS["c2_base_itc_bf16"]
    q, k, v = synth.make_qkv(wl)
    out, lse = _run(wl, q, k, v, None)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    # every (batch, head) slice, head-major so that the oracle builds each head's mask once
    _compare(wl, q, k, v, None, out, lse, slices=[(bi, h) for h in range(wl.H) for bi in range(wl.B)])


def test_c2_full_size_closed_forms():
    """Properties that hold at any size, on the full BigBird-base workload: V == 1 gives out == 1 everywhere;
    Q == 0 gives lse = ln(64 * attended key blocks) per row, and the block counts are those of the layout."""
    wl = synth.WORKLOADS["c2_base_itc_bf16"]
    q, k, v = synth.make_qkv(wl)
    out, _ = _run(wl, q, k, torch.ones_like(v), None)
    assert np.abs(out - 1).max() <= 2 ** -8
    out, lse = _run(wl, torch.zeros_like(q), k, v, None)
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    rp, _ = L.export()
    blocks = np.diff(rp).reshape(wl.H, wl.nb)                      # attended key blocks per (head, query block)
    want = np.log(64.0 * np.repeat(blocks, 64, axis=1))            # [H, N]
    assert np.abs(lse - want[None]).max() < 1e-4
    L.close()
    # a key block permuted inside itself, jointly in K and V, changes nothing
    perm = torch.arange(wl.N).reshape(wl.nb, 64)[:, torch.randperm(64, generator=torch.Generator().manual_seed(0))].reshape(-1)
    a, la = _run(wl, q, k, v, None)
    b2, lb = _run(wl, q, k[:, :, perm], v[:, :, perm], None)
    assert np.abs(a - b2).max() <= 2e-2 and np.abs(la - lb).max() <= 1e-4


def test_c3_etc_bf16_full_size():
    wl = synth.WORKLOADS["c3_etc_bf16"]
    q, k, v = synth.make_qkv(wl)
    out, lse = _run(wl, q, k, v, None)
    assert np.isfinite(out).all() and np.isfinite(lse).all()
    _compare(wl, q, k, v, None, out, lse, slices=[(bi, h) for h in range(wl.H) for bi in range(wl.B)])


def test_c4_long_itc_bf16_full_size():
    wl = synth.WORKLOADS["c4_long_itc_bf16"]
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    out, lse = _run(wl, q, k, v, kpm)
    rng = np.random.default_rng(1)
    rows = np.unique(np.concatenate([
        np.arange(0, 64), np.arange(wl.N - 64, wl.N),            # the global query blocks (the last one is padding)
        np.arange(12928, 13056),                                  # around the valid length 13000
        rng.choice(wl.N, size=320, replace=False)]))
    _compare(wl, q, k, v, kpm, out, lse, slices=[(0, h) for h in range(0, wl.H, 2)], rows=rows)
    pad = kpm[0].numpy() == 0
    assert (out[0][:, pad] == 0).all() and np.isneginf(lse[0][:, pad]).all()
    assert np.isfinite(out).all() and np.isfinite(lse[0][:, ~pad]).all()


def test_c5_large_ragged_bf16_full_size():
    wl = synth.WORKLOADS["c5_large_ragged_bf16"]
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    lens = synth.valid_lengths(wl)
    out, lse = _run(wl, q, k, v, kpm)
    shortest, longest = int(np.argmin(lens)), int(np.argmax(lens))
    slices = sorted(set([(shortest, 0), (shortest, wl.H - 1), (longest, 3), (longest, 8)] + _sample_slices(wl, 4, seed=2)))
    _compare(wl, q, k, v, kpm, out, lse, slices=slices)
    assert np.isfinite(out).all()
    for bi in range(wl.B):
        assert (out[bi][:, lens[bi]:] == 0).all() and np.isneginf(lse[bi][:, lens[bi]:]).all()
        assert np.isfinite(lse[bi][:, : lens[bi]]).all()
