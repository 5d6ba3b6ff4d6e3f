"""Pins for the fp64 oracle: it is checked against what the paper and the mathematics
fix, never against itself and never against the CUDA path.

Citations are to arXiv 2007.14062: Sec. 2 (Eq. AT, adjacency matrix A, random /
window / global attention, ITC and ETC), App. D (block-sparse definitions, the
12-token example with block size 2, the cost O(n(g+w+r)bd)).
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import logsumexp

from oracle import bigbird_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden_lines(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.strip() for ln in f if ln.strip() and not ln.startswith("#")]


# ----------------------------------------------------------------------------- generator
def test_splitmix64_published_vectors():
    want = [int(x, 16) for x in _golden_lines("splitmix64_state0.txt")]
    s, got = 0, []
    for _ in want:
        s, z = O.splitmix64_next(s)
        got.append(z)
    assert got == want


def test_stream_key_separates_seed_head_block():
    keys = {O.stream_key(s, h, j) for s in range(4) for h in range(16) for j in range(256)}
    assert len(keys) == 4 * 16 * 256
    assert O.stream_key(0, 0, 0) == 0
    assert O.stream_key(1, 0, 0) == 1 << 40
    assert O.stream_key(0, 1, 0) == 1 << 20
    assert O.stream_key(0, 0, 1) == 1


def _random_block_vectors():
    out = []
    for ln in _golden_lines("random_blocks_seed0.txt"):
        lhs, rhs = ln.split(":")
        nb, w, g, r, seed, h, j = (int(x) for x in lhs.split())
        out.append((nb, w, g, r, seed, h, j, [int(x) for x in rhs.split()]))
    return out


def test_random_blocks_hand_worked_vectors():
    """App. D item 1 under the written generator spec: selections worked by hand from SplitMix64's
    published outputs (derivation in the golden file).  A different bounded draw (z mod m), a shuffle
    from the far end or a draw with replacement gives other blocks."""
    vecs = _random_block_vectors()
    assert len(vecs) >= 3
    for nb, w, g, r, seed, h, j, want in vecs:
        for b in (1, 4):
            assert O.random_blocks(O.Graph(nb * b, b, w, g, r, seed, h + 1, O.ITC), h, j) == want


# ----------------------------------------------------------------------------- block sets
def _params():
    out = []
    for nb, b, w, g, r, mode in itertools.product([4, 6, 8, 13, 64], [1, 2, 4], [1, 3, 5], [0, 1, 2, 3],
                                                  [0, 1, 3], [O.ITC, O.ETC]):
        if g > nb:
            continue
        out.append(O.Graph(nb * b, b, w, g, r, 7, 2, mode))
    return out


def test_random_blocks_invariants():
    """App. D item 1: exactly r random key blocks per query block (all candidates if fewer),
    none of them in the window or global, none repeated; global query blocks draw nothing."""
    for gr in _params():
        G = set(O.global_blocks(gr))
        for h in range(gr.H):
            for j in range(gr.nb):
                R = O.random_blocks(gr, h, j)
                assert R == sorted(set(R))
                if j in G:
                    assert R == []
                    continue
                W = set(O.window_blocks(gr, j))
                cand = set(range(gr.nb)) - G - W
                assert set(R) <= cand
                assert len(R) == min(gr.r, len(cand))


def test_random_blocks_are_uniform_over_candidates():
    """Each candidate is chosen with probability r/m (sampling without replacement)."""
    gr = O.Graph(24 * 4, 4, 3, 2, 3, 11, 400, O.ITC)
    j = 10
    cand = [c for c in range(gr.nb) if c not in O.global_blocks(gr) and c not in O.window_blocks(gr, j)]
    counts = dict.fromkeys(cand, 0)
    for h in range(gr.H):
        for c in O.random_blocks(gr, h, j):
            counts[c] += 1
    m = len(cand)
    p = gr.r / m
    sd = math.sqrt(gr.H * p * (1 - p))
    for c in cand:
        assert abs(counts[c] - gr.H * p) < 4.5 * sd, (c, counts[c], gr.H * p)
    # heads, blocks and seeds get different draws
    assert len({tuple(O.random_blocks(gr, h, j)) for h in range(50)}) > 25
    gr2 = O.Graph(gr.N, gr.b, gr.w, gr.g, gr.r, 12, gr.H, gr.mode)
    assert any(O.random_blocks(gr, h, j) != O.random_blocks(gr2, h, j) for h in range(8))


def test_global_and_window_sets():
    gr = O.Graph(64 * 8, 8, 3, 2, 3, 0, 1, O.ITC)
    assert O.global_blocks(gr) == [0, 63]                       # first and last
    assert O.global_blocks(O.Graph(64, 8, 3, 3, 0, 0, 1, O.ITC)) == [0, 1, 7]
    assert O.global_blocks(O.Graph(64, 8, 3, 3, 0, 0, 1, O.ETC)) == [0, 1, 2]
    assert O.window_blocks(gr, 5) == [4, 5, 6]                  # App. D item 2
    assert O.window_blocks(gr, 0) == [0, 1]                     # clipped, no wrap-around
    assert O.window_blocks(gr, 63) == [62, 63]
    assert O.window_blocks(O.Graph(64, 8, 5, 0, 0, 0, 1), 3) == [1, 2, 3, 4, 5]


# ----------------------------------------------------------------------------- adjacency matrix
def test_mask_structure_matches_definitions():
    """Sec. 2: A(i,:) = A(:,i) = 1 for i in G; window band; every other 1 is a random block."""
    for gr in _params():
        if gr.nb > 13:
            continue
        G = O.global_blocks(gr)
        hw = (gr.w - 1) // 2
        for h in range(gr.H):
            A = O.build_mask(gr, h)
            assert A.shape == (gr.N, gr.N) and A.dtype == bool
            blk = A.reshape(gr.nb, gr.b, gr.nb, gr.b)
            # constant inside every b x b block (App. D: parameters act on blocks as units)
            assert (blk == blk[:, :1, :, :1]).all()
            Ab = blk[:, 0, :, 0]
            for Gi in G:
                assert Ab[Gi, :].all() and Ab[:, Gi].all()
            for I in range(gr.nb):
                for C in range(gr.nb):
                    if abs(I - C) <= hw:
                        assert Ab[I, C]
                if I in G:
                    continue
                extra = [C for C in range(gr.nb) if Ab[I, C] and abs(I - C) > hw and C not in G]
                assert extra == O.random_blocks(gr, h, I)
                cand = gr.nb - len(set(G) | set(O.window_blocks(gr, I)))
                assert Ab[I].sum() == len(set(G) | set(O.window_blocks(gr, I))) + min(gr.r, cand)


def test_pairs_per_head_match_hand_counts():
    for ln in _golden_lines("pairs_per_head.txt"):
        name, nb, mode, r, pairs = ln.split()
        nb, mode, r, pairs = int(nb), int(mode), int(r), int(pairs)
        gr = O.Graph(nb * 2, 2, 3, 2, r, 5, 2, mode)
        row_ptr, col_idx = O.layout_from_mask(gr)
        per_head = np.diff(row_ptr).reshape(gr.H, nb).sum(axis=1)
        assert (per_head == pairs).all(), (name, per_head)
        # App. D cost formula: a sparse row never lists more than g+w+r blocks
        G = O.global_blocks(gr)
        cnt = np.diff(row_ptr).reshape(gr.H, nb)
        for I in range(nb):
            if I in G:
                assert (cnt[:, I] == nb).all()
            else:
                assert (cnt[:, I] <= gr.g + gr.w + gr.r).all()
        interior = [I for I in range(3, nb - 3)]
        assert (cnt[:, interior] == (2 + 3 + r)).all()


def test_tiny_config_degenerate_structure():
    """nb=8, w=3, g=2, r=3: rows 2..5 have exactly 3 candidates so they attend all 8 blocks
    whatever the seed; rows 1 and 6 take 3 of 4 candidates, so exactly one block is missing."""
    for seed in range(5):
        gr = O.Graph(512, 64, 3, 2, 3, seed, 2, O.ITC)
        row_ptr, _ = O.layout_from_mask(gr)
        cnt = np.diff(row_ptr).reshape(2, 8)
        assert (cnt == np.array([8, 7, 8, 8, 8, 8, 7, 8])).all()


def test_etc_matrix_B_is_shifted_A_plus_global_rows_and_columns():
    """Sec. 2, ETC: B(i,:) = B(:,i) = 1 for the g added tokens and B(g+i, g+j) = A(i,j)."""
    b, nb_seq, gblk = 2, 9, 2
    A = O.build_mask(O.Graph(nb_seq * b, b, 3, 0, 0, 0, 1, O.ITC), 0)        # window-only graph on N tokens
    Bm = O.build_mask(O.Graph((nb_seq + gblk) * b, b, 3, gblk, 0, 0, 1, O.ETC), 0)
    gt = gblk * b
    assert Bm[:gt, :].all() and Bm[:, :gt].all()
    # in the first sequence block the window reaches back into the global block, which is 1 anyway
    assert (Bm[gt:, gt:] == A).all()


def test_mask_is_a_directed_graph():
    """Random edges are per query block and not symmetrised: A differs from its transpose,
    while the window+global part alone is symmetric (catches a transposed mask)."""
    gr = O.Graph(32 * 2, 2, 3, 2, 3, 3, 1, O.ITC)
    A = O.build_mask(gr, 0)
    assert not (A == A.T).all()
    A0 = O.build_mask(O.Graph(gr.N, gr.b, gr.w, gr.g, 0, 3, 1, O.ITC), 0)
    assert (A0 == A0.T).all()
    # rows (not columns) carry exactly r extra blocks
    extra = (A & ~A0).reshape(gr.nb, gr.b, gr.nb, gr.b)[:, 0, :, 0]
    sparse_rows = [I for I in range(gr.nb) if I not in O.global_blocks(gr)]
    assert (extra[sparse_rows].sum(axis=1) == 3).all()
    assert len(set(extra.sum(axis=0).tolist())) > 1


# ----------------------------------------------------------------------------- attention values
def _rng_qkv(N, D, seed):
    rng = np.random.default_rng(seed)
    return rng.standard_normal((N, D)), rng.standard_normal((N, D)), rng.standard_normal((N, D))


def _neighbours(gr, h, i):
    """Out-neighbour set N(i) of token i, from the block-level sentences of App. D,
    written with sets and loops (independent of the oracle's mask construction)."""
    I = i // gr.b
    if gr.mode == O.ETC:
        G = set(range(gr.g))
    else:
        G = set(range((gr.g + 1) // 2)) | set(range(gr.nb - gr.g // 2, gr.nb))
    if I in G:
        blocks = set(range(gr.nb))
    else:
        half = (gr.w - 1) // 2
        blocks = {c for c in range(I - half, I + half + 1) if 0 <= c < gr.nb} | G
        blocks |= set(O.random_blocks(gr, h, I))
    return sorted(k for c in blocks for k in range(c * gr.b, (c + 1) * gr.b))


@pytest.mark.parametrize("N,b,w,g,r,mode", [
    (12, 2, 3, 1, 1, O.ITC),     # App. D worked example: 12 tokens, block size 2, r=1, w=3, g=1
    (12, 1, 3, 2, 2, O.ITC),     # Fig. 1 caption: token level, r=2, w=3, g=2
    (16, 2, 3, 2, 1, O.ETC),
    (24, 4, 5, 2, 2, O.ITC),
])
def test_brute_force_eq_AT_on_tiny_graphs(N, b, w, g, r, mode):
    """Eq. (AT) evaluated neighbour by neighbour in Python loops equals the masked-dense oracle."""
    gr = O.Graph(N, b, w, g, r, 21, 2, mode)
    D = 5
    scale = 0.37
    for h in range(gr.H):
        q, k, v = _rng_qkv(N, D, 100 + h)
        A = O.build_mask(gr, h)
        out, lse = O.attend(q, k, v, A, None, scale)
        for i in range(N):
            nbrs = _neighbours(gr, h, i)
            assert sorted(np.nonzero(A[i])[0].tolist()) == nbrs
            s = [scale * sum(q[i, u] * k[j, u] for u in range(D)) for j in nbrs]
            mx = max(s)
            e = [math.exp(x - mx) for x in s]
            tot = sum(e)
            want = [sum(e[t] / tot * v[j, u] for t, j in enumerate(nbrs)) for u in range(D)]
            assert np.allclose(out[i], want, rtol=0, atol=1e-12)
            assert abs(lse[i] - (mx + math.log(tot))) < 1e-12


@pytest.mark.parametrize("how", ["wide_window", "all_global"])
def test_complete_digraph_recovers_full_attention(how):
    """Sec. 2: if D is the complete digraph the mechanism is full quadratic attention.
    Compared with library routines (torch SDPA in fp64, scipy logsumexp)."""
    nb, b, Dh = 6, 4, 8
    if how == "wide_window":
        gr = O.Graph(nb * b, b, 2 * nb - 1, 0, 0, 0, 1, O.ITC)
    else:
        gr = O.Graph(nb * b, b, 1, nb, 0, 0, 1, O.ITC)
    A = O.build_mask(gr, 0)
    assert A.all()
    q, k, v = _rng_qkv(gr.N, Dh, 5)
    scale = 1 / math.sqrt(Dh)
    out, lse = O.attend(q, k, v, A, None, scale)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None], scale=scale)[0].numpy()
    assert np.abs(out - ref).max() < 1e-13
    assert np.abs(lse - logsumexp(scale * q @ k.T, axis=1)).max() < 1e-13


def test_closed_forms():
    gr = O.Graph(16 * 4, 4, 3, 2, 3, 9, 1, O.ITC)
    A = O.build_mask(gr, 0)
    q, k, v = _rng_qkv(gr.N, 6, 1)
    valid = np.ones(gr.N, dtype=bool)
    valid[50:] = False
    # V == 1  =>  out == 1 (softmax weights sum to one)
    out, _ = O.attend(q, k, np.ones_like(v), A, valid, 0.5)
    assert np.abs(out - 1).max() < 1e-14
    # Q == 0  =>  uniform weights: out = mean of attended valid V rows, lse = ln(count)
    out, lse = O.attend(np.zeros_like(q), k, v, A, valid, 0.5)
    keep = A & valid[None, :]
    cnt = keep.sum(axis=1)
    assert np.abs(lse - np.log(cnt)).max() < 1e-14
    assert np.abs(out - (keep.astype(float) @ v) / cnt[:, None]).max() < 1e-14
    # an interior row of the 4096-token base config sees (3+2+3)*64 = 512 keys
    big = O.Graph(4096, 64, 3, 2, 3, 1, 1, O.ITC)
    assert O.mask_rows(big, 0, [64 * 30 + 5]).sum() == 512
    # adding a constant to every score of a row shifts lse and leaves out unchanged
    q2 = np.concatenate([q, np.ones((gr.N, 1))], axis=1)
    k2 = np.concatenate([k, 3.0 * np.ones((gr.N, 1))], axis=1)
    o1, l1 = O.attend(q, k, v, A, valid, 0.5)
    o2, l2 = O.attend(q2, k2, v, A, valid, 0.5)
    assert np.abs(o1 - o2).max() < 1e-13 and np.abs(l2 - l1 - 1.5).max() < 1e-13
    # one-hot block V: column c of the result is the attention mass on key block c;
    # it is exactly zero for blocks outside the row's list and the masses sum to one
    onehot = np.zeros((gr.N, gr.nb))
    onehot[np.arange(gr.N), np.arange(gr.N) // gr.b] = 1
    mass, _ = O.attend(q, k, onehot, A, None, 0.5)
    Ab = A.reshape(gr.nb, gr.b, gr.nb, gr.b)[:, 0, :, 0]
    rows_blk = np.arange(gr.N) // gr.b
    assert (mass[~Ab[rows_blk]] == 0).all() and (mass[Ab[rows_blk]] > 0).all()
    assert np.abs(mass.sum(axis=1) - 1).max() < 1e-14


def test_key_order_inside_a_block_does_not_matter():
    gr = O.Graph(10 * 4, 4, 3, 2, 2, 2, 1, O.ITC)
    A = O.build_mask(gr, 0)
    q, k, v = _rng_qkv(gr.N, 6, 2)
    perm = np.arange(gr.N).reshape(gr.nb, gr.b)[:, ::-1].reshape(-1)     # reverse inside each block
    o1, l1 = O.attend(q, k, v, A, None, 0.4)
    o2, l2 = O.attend(q, k[perm], v[perm], A, None, 0.4)
    assert np.abs(o1 - o2).max() < 1e-13 and np.abs(l1 - l2).max() < 1e-13


def test_padding_equals_truncation():
    """Masking keys >= L equals running on sequences cut to L with the same graph
    restricted to the first L tokens."""
    gr = O.Graph(12 * 4, 4, 3, 2, 2, 4, 1, O.ITC)
    A = O.build_mask(gr, 0)
    q, k, v = _rng_qkv(gr.N, 6, 3)
    for L in (gr.N, 30, 17, 4):
        valid = np.arange(gr.N) < L
        o1, l1 = O.attend(q, k, v, A, valid, 0.4)
        o2, l2 = O.attend(q[:L], k[:L], v[:L], A[:L, :L], None, 0.4)
        assert np.abs(o1[:L] - o2).max() < 1e-13 and np.abs(l1[:L] - l2).max() < 1e-13
    # a row with no valid attended key: out = 0, lse = -inf, no NaN
    o, l = O.attend(q, k, v, A, np.zeros(gr.N, dtype=bool), 0.4)
    assert (o == 0).all() and np.isneginf(l).all()


def test_attention_wrapper_slices_and_rows():
    gr = O.Graph(8 * 4, 4, 3, 2, 1, 6, 2, O.ITC)
    rng = np.random.default_rng(0)
    q, k, v = (rng.standard_normal((2, 2, gr.N, 4)) for _ in range(3))
    kpm = np.ones((2, gr.N), dtype=np.uint8)
    kpm[1, 20:] = 0
    full = O.attention(q, k, v, gr, kpm, 0.5)
    assert set(full) == {(0, 0), (0, 1), (1, 0), (1, 1)}
    part = O.attention(q, k, v, gr, kpm, 0.5, slices=[(1, 1)], rows=[3, 9])
    assert np.array_equal(part[(1, 1)][0], full[(1, 1)][0][[3, 9]])
    want, _ = O.attend(q[1, 1], k[1, 1], v[1, 1], O.build_mask(gr, 1), kpm[1] != 0, 0.5)
    assert np.array_equal(full[(1, 1)][0], want)


def test_graph_rejects_bad_parameters():
    for bad in [dict(N=10, b=4), dict(w=2), dict(g=99), dict(r=-1), dict(mode=3), dict(H=0), dict(seed=1 << 24), dict(seed=-1)]:
        kw = dict(N=16, b=4, w=3, g=2, r=1, seed=0, H=1, mode=0)
        kw.update(bad)
        with pytest.raises(ValueError):
            O.Graph(**kw)


# ----------------------------------------------------------------------------- gradients
def _loss(q, k, v, A, kv, scale, dout, rv=None):
    out, _ = O.attend(q, k, v, A, kv, scale)
    if rv is not None:
        out = out * rv[:, None]
    return float((out * dout).sum())


@pytest.mark.parametrize("N,b,w,g,r,mode", [(12, 2, 3, 1, 1, O.ITC), (16, 1, 3, 2, 2, O.ITC), (14, 2, 3, 2, 0, O.ETC)])
def test_gradients_match_central_differences_of_the_forward_oracle(N, b, w, g, r, mode):
    """dq, dk, dv of `attend_bwd` against central finite differences of sum(out * dout) computed with the forward
    oracle on the paper's toy sizes (App. D: 12 tokens, block 2; Fig. 1: token level), with padded keys and a
    padded query row.  A dropped term, a wrong sign or a transposed operand shows up here."""
    gr = O.Graph(N, b, w, g, r, 3, 1, mode)
    rng = np.random.default_rng(N)
    D = 4
    q, k, v, dout = (rng.standard_normal((N, D)) for _ in range(4))
    kv = np.ones(N, dtype=bool)
    kv[-3:] = False
    A = O.build_mask(gr, 0)
    scale = 0.7
    dq, dk, dv = O.attend_bwd(q, k, v, A, kv, scale, dout, row_valid=kv)
    eps = 1e-6
    for name, x, g_ in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        num = np.zeros_like(x)
        for idx in np.ndindex(*x.shape):
            old = x[idx]
            x[idx] = old + eps
            fp = _loss(q, k, v, A, kv, scale, dout, kv.astype(float))
            x[idx] = old - eps
            fm = _loss(q, k, v, A, kv, scale, dout, kv.astype(float))
            x[idx] = old
            num[idx] = (fp - fm) / (2 * eps)
        assert np.abs(num - g_).max() < 1e-7, name
    assert (dq[~kv] == 0).all()                       # a padded query row gets no gradient
    assert np.abs(dk[~kv]).max() == 0 and np.abs(dv[~kv]).max() == 0      # a padded key gets none either


def test_gradients_on_the_complete_digraph_match_autograd_through_sdpa():
    """Sec. 2: on the complete digraph Eq. (AT) is full attention, so the gradients must be those torch's
    autograd computes through scaled_dot_product_attention in fp64."""
    N, D = 24, 8
    gr = O.Graph(N, 4, 2 * (N // 4) - 1, 0, 0, 0, 1, O.ITC)
    A = O.build_mask(gr, 0)
    assert A.all()
    rng = np.random.default_rng(5)
    q, k, v, dout = (rng.standard_normal((N, D)) for _ in range(4))
    scale = 1.0 / math.sqrt(D)
    dq, dk, dv = O.attend_bwd(q, k, v, A, None, scale, dout)
    tq, tk, tv = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v))
    out = torch.nn.functional.scaled_dot_product_attention(tq[None, None], tk[None, None], tv[None, None], scale=scale)[0, 0]
    (out * torch.tensor(dout)).sum().backward()
    assert np.abs(tq.grad.numpy() - dq).max() < 1e-12
    assert np.abs(tk.grad.numpy() - dk).max() < 1e-12
    assert np.abs(tv.grad.numpy() - dv).max() < 1e-12


def test_gradient_closed_forms_and_wrapper():
    """Q == 0 makes every row uniform over its attended keys: dk == 0 and dv[key] = sum over the rows attending
    it of dout[row] / (number of keys the row attends).  The wrapper loops (batch, head) slices over attend_bwd."""
    gr = O.Graph(32, 4, 3, 2, 1, 1, 2, O.ITC)
    rng = np.random.default_rng(9)
    B, D = 2, 4
    q = np.zeros((B, gr.H, gr.N, D))
    k, v, dout = (rng.standard_normal((B, gr.H, gr.N, D)) for _ in range(3))
    res = O.attention_bwd(q, k, v, dout, gr, None, 0.5)
    for (bi, h), (dq, dk, dv) in res.items():
        A = O.build_mask(gr, h).astype(np.float64)
        W = A / A.sum(axis=1, keepdims=True)
        assert np.abs(dk).max() < 1e-15
        assert np.abs(dv - W.T @ dout[bi, h]).max() < 1e-13
        want = O.attend_bwd(q[bi, h], k[bi, h], v[bi, h], O.build_mask(gr, h), None, 0.5, dout[bi, h])
        assert all(np.array_equal(a, b) for a, b in zip((dq, dk, dv), want))
