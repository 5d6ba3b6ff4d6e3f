"""Host-side checks of the library's layout builder against the oracle's token-level mask (bit-exact),
and of the tile schedule derived from it.  No GPU needed."""
import ctypes as C
import itertools

import numpy as np
import pytest

import paper_2007_14062_b200 as bb
from paper_2007_14062_b200 import synth
from oracle import bigbird_oracle as O


def _oracle_csr(N, b, w, g, r, seed, H, mode):
    return O.layout_from_mask(O.Graph(N, b, w, g, r, seed, H, mode))


SWEEP = [(nb * b, b, w, g, r, seed, H, mode)
         for nb, b, w, g, r, seed, H, mode in itertools.product(
             [1, 2, 3, 5, 8, 13, 31], [1, 2, 64], [1, 3, 5, 7], [0, 1, 2, 3, 5], [0, 1, 3, 6], [0, 9], [1, 3], [0, 1])
         if g <= nb]


def test_layout_sweep_bit_exact():
    rng = np.random.default_rng(0)
    picks = rng.choice(len(SWEEP), size=400, replace=False)
    for i in picks:
        N, b, w, g, r, seed, H, mode = SWEEP[i]
        L = bb.bigbird_build_layout(N, b, w, g, r, seed, H, mode)
        rp, ci = L.export()
        orp, oci = _oracle_csr(N, b, w, g, r, seed, H, mode)
        assert np.array_equal(rp, orp), SWEEP[i]
        assert np.array_equal(ci, oci), SWEEP[i]
        L.close()


@pytest.mark.parametrize("cfg", [(84 * (3 + 49), 84, 3, 3, 0, 0, 12, 1),      # ETC base: block 84, 4116 tokens + 3 global blocks
                                 (169 * (3 + 24), 169, 3, 3, 0, 0, 16, 1),    # QA large: block 169, 4056 tokens + 3 global blocks
                                 (84 * 49, 84, 3, 2, 3, 5, 4, 0)])            # the same block size with random blocks, ITC
def test_layout_of_the_papers_etc_block_sizes_bit_exact(cfg):
    """Block sizes of the paper's ETC settings (App. E hyper-parameter tables): the graph is built in blocks, so only
    N % b == 0 matters; the global token count is rounded up to whole blocks by the caller and the tail masked."""
    L = bb.bigbird_build_layout(*cfg)
    rp, ci = L.export()
    orp, oci = _oracle_csr(*cfg)
    assert np.array_equal(rp, orp) and np.array_equal(ci, oci)
    cp, ri = L.export_transposed()
    assert cp[-1] == rp[-1] and len(ri) == len(ci)
    L.close()


def test_library_random_blocks_match_hand_worked_vectors():
    """The library's own selection against the hand-worked vectors of tests/golden/random_blocks_seed0.txt
    (App. D item 1 under the generator spec of bigbird.h), independently of the oracle."""
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "random_blocks_seed0.txt")
    n = 0
    for ln in open(path):
        if not ln.strip() or ln.startswith("#"):
            continue
        lhs, rhs = ln.split(":")
        nb, w, g, r, seed, h, j = (int(x) for x in lhs.split())
        want = [int(x) for x in rhs.split()]
        hw = (w - 1) // 2
        window = [c for c in range(j - hw, j + hw + 1) if 0 <= c < nb]
        L = bb.bigbird_build_layout(nb * 2, 2, w, g, r, seed, h + 1, bb.BIGBIRD_ITC)
        rp, ci = L.export()
        row = h * nb + j
        assert list(ci[rp[row]:rp[row + 1]]) == sorted(set(window) | set(want)), ln
        L.close()
        n += 1
    assert n >= 3


@pytest.mark.parametrize("name", synth.ORDER)
def test_layout_of_the_five_workloads_bit_exact(name):
    wl = synth.WORKLOADS[name]
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    rp, ci = L.export()
    orp, oci = _oracle_csr(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    assert rp.dtype == np.int32 and ci.dtype == np.int32
    assert np.array_equal(rp, orp) and np.array_equal(ci, oci)
    per_head = np.diff(rp).reshape(wl.H, wl.nb).sum(axis=1)
    want = {"c1_tiny_itc_fp32": 62, "c2_base_itc_bf16": 622, "c3_etc_bf16": 450, "c4_long_itc_bf16": 2542,
            "c5_large_ragged_bf16": 622}[name]
    assert (per_head == want).all()


def test_transposed_lists_are_the_transpose_of_the_oracle_mask():
    """Row (h, c) of the transposed export lists, ascending, the query blocks whose oracle mask attends key block c."""
    for cfg in [(512, 64, 3, 2, 3, 0, 2, 0), (4224, 64, 3, 2, 0, 2, 2, 1), (13 * 4, 4, 5, 3, 2, 5, 3, 0), (6, 1, 3, 6, 0, 0, 1, 1),
                (7 * 2, 2, 3, 0, 6, 1, 2, 0)]:
        N, b, w, g, r, seed, H, mode = cfg
        nb = N // b
        L = bb.bigbird_build_layout(*cfg)
        cp, ri = L.export_transposed()
        assert cp.dtype == np.int32 and ri.dtype == np.int32 and cp[0] == 0 and cp[-1] == L.nnz
        gr = O.Graph(N, b, w, g, r, seed, H, mode)
        first = np.arange(nb) * b
        for h in range(H):
            A = O.mask_rows(gr, h, first)[:, first]                  # block-level adjacency [query block, key block]
            for c in range(nb):
                got = ri[cp[h * nb + c]:cp[h * nb + c + 1]]
                assert list(got) == list(np.nonzero(A[:, c])[0]), (cfg, h, c)
        L.close()


def test_window_choice_is_moot_for_the_five_workloads():
    """With w=3 a circular window would only add blocks that are global anyway (first/last rows in ITC,
    block 0 in ETC), so clipped and circular windows give the same graph on all five workloads."""
    for wl in synth.WORKLOADS.values():
        G = set(O.global_blocks(O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, 1, wl.mode)))
        hw = (wl.w - 1) // 2
        for j in range(wl.nb):
            wrapped = {(j + d) % wl.nb for d in range(-hw, hw + 1)}
            clipped = {c for c in range(j - hw, j + hw + 1) if 0 <= c < wl.nb}
            assert j in G or (wrapped - clipped) <= G


@pytest.mark.parametrize("cfg", [(512, 64, 3, 2, 3, 0, 2, 0), (4096, 64, 3, 2, 3, 1, 3, 0), (4224, 64, 3, 2, 0, 2, 2, 1),
                                 (13 * 4, 4, 5, 3, 2, 5, 2, 0), (7 * 2, 2, 3, 1, 6, 1, 2, 1), (3, 1, 1, 0, 0, 0, 1, 0),
                                 (6, 1, 3, 6, 0, 0, 1, 1)])
def test_schedule_covers_every_listed_pair_exactly_once(cfg):
    N, b, w, g, r, seed, H, mode = cfg
    L = bb.bigbird_build_layout(*cfg)
    rp, ci = L.export()
    nb = N // b
    sizes, items, base, steps = L.schedule()
    ipH, heavy = int(sizes[0]), int(sizes[1])
    assert sizes[3] == H and items.shape == (H * ipH, 8)
    for h in range(H):
        seen = {}
        for it in items[h * ipH:(h + 1) * ipH]:
            qa, qb, sbeg, scnt, part, nparts, tile, _ = (int(x) for x in it)
            assert 0 <= qa < nb and (qb == -1 or 0 <= qb < nb) and qa != qb
            for s in steps[base[h] + sbeg: base[h] + sbeg + scnt]:
                c, who = int(s[0]), int(s[1])
                assert 0 <= c < nb and who in (0, 1, 2)
                assert qb >= 0 or who == 0
                pairs = ([(qa, c)] if who in (0, 1) else []) + ([(qb, c)] if who in (0, 2) and qb >= 0 else [])
                for pr in pairs:
                    assert pr not in seen
                    seen[pr] = 1
        want = {(j, int(c)) for j in range(nb) for c in ci[rp[h * nb + j]: rp[h * nb + j + 1]]}
        assert set(seen) == want
        # heavy items come first and are exactly the global query blocks
        G = set(O.global_blocks(O.Graph(N, b, w, g, r, seed, H, mode)))
        hq = {int(x) for it in items[h * ipH: h * ipH + heavy] for x in it[:2] if x >= 0}
        assert hq == G


def test_bad_arguments_return_error_codes():
    lib = bb.lib()
    h = C.c_void_p(None)
    bad = [
        (100, 64, 3, 2, 3, 0, 1, 0),     # N % b != 0
        (512, 64, 2, 2, 3, 0, 1, 0),     # even window
        (512, 64, 3, 9, 3, 0, 1, 0),     # more global blocks than blocks
        (512, 64, 3, 2, -1, 0, 1, 0),
        (512, 64, 3, 2, 3, 0, 0, 0),     # no heads
        (512, 64, 3, 2, 3, 0, 1, 7),     # unknown mode
        (0, 64, 3, 2, 3, 0, 1, 0),
        (512, 0, 3, 2, 3, 0, 1, 0),
        (512, 64, 3, 2, 3, 1 << 30, 1, 0),   # seed does not fit the stream key
    ]
    for args in bad:
        assert lib.bigbird_build_layout(*args, C.byref(h)) == -1, args
        assert h.value is None
    assert lib.bigbird_build_layout(512, 64, 3, 2, 3, 0, 1, 0, None) == -1
    n = C.c_int64(0)
    assert lib.bigbird_layout_nnz(None, C.byref(n)) == -1
    assert lib.bigbird_layout_export(None, None, None) == -1
    assert lib.bigbird_layout_destroy(None) == -1
    assert lib.bigbird_last_status(None, None, None) == -1
    # attention entry points validate before touching the GPU
    L = bb.bigbird_build_layout(512, 64, 3, 2, 3, 0, 2, 0)
    for fn in (lib.bigbird_attn_fwd, lib.bigbird_attn_fwd_simt):
        assert fn(None, None, None, L.handle, None, None, None, 1, 2, 512, 64, 64, 0.125, 0, None) == -1
        fake = C.c_void_p(4096)
        assert fn(fake, fake, fake, L.handle, None, fake, None, 1, 2, 1024, 64, 64, 0.125, 0, None) == -1   # other N
        assert fn(fake, fake, fake, L.handle, None, fake, None, 1, 3, 512, 64, 64, 0.125, 0, None) == -1    # other H
        assert fn(fake, fake, fake, L.handle, None, fake, None, 1, 2, 512, 64, 64, 0.125, 5, None) == -2    # dtype
        assert fn(fake, fake, fake, L.handle, None, fake, None, 1, 2, 512, 48, 64, 0.125, 0, None) == -2    # D
        assert fn(C.c_void_p(4100), fake, fake, L.handle, None, fake, None, 1, 2, 512, 64, 64, 0.125, 0, None) == -1
    assert bb.bigbird_strerror(-1) == "invalid argument" and bb.bigbird_strerror(0) == "ok"
    with pytest.raises(bb.BigBirdError):
        bb.bigbird_build_layout(100, 64, 3, 2, 3, 0, 1, 0)
