"""fp64 CPU oracle for BigBird block-sparse attention (TEST INFRASTRUCTURE).

This file is the slow, plain statement of what the CUDA library must compute.
It is used only by the tests, by the smoke check and by the benchmark's CPU
baseline leg.  The library never imports it and shares no code with it.

What it states (arXiv 2007.14062):

* Sec. 2, Eq. (AT): output i = sum over the out-neighbours N(i) of
  softmax(q_i . k_j) v_j, per head.  Only the per-head softmax-attention core
  is in scope here: no residual x_i, no sum over heads, no projections.  The
  scoring function sigma is softmax; the 1/sqrt(d) factor the equation leaves
  out is the explicit `scale` argument.
* Sec. 2: adjacency matrix A, A(i, j) = 1 iff query i attends to key j;
  random attention (r keys per query), sliding window (w/2 to each side) and
  global tokens (A(i, :) = A(:, i) = 1 for i in G), in the ITC flavour (existing
  tokens are global) and the ETC flavour (extra tokens are prepended; matrix B).
* App. D ("Implementation details"): the same three families on b x b blocks:
  query block j attends key blocks j-(w-1)/2 .. j+(w-1)/2, r random key blocks
  and the g global blocks; global query blocks attend everything.

Readings taken where the paper is silent (each is a deliberate choice):

* w, g, r are given in BLOCKS; w is odd.
* ITC global set: the first ceil(g/2) and the last floor(g/2) blocks.  ETC global
  set: the first g blocks of the (extended) sequence.
* The window is clipped at the sequence ends (no wrap-around).
* Random blocks: per (head, query block), the same for every batch element,
  drawn WITHOUT replacement from the ascending list of blocks that are neither
  in the query block's window nor global; if there are fewer than r such
  blocks all are taken; global query blocks draw nothing.
* The generator is not specified by the paper.  Here: a SplitMix64 stream
  (Steele, Lea, Flood 2014; Vigna's public-domain constants) whose initial
  state is (seed << 40) ^ (h << 20) ^ j, a bounded draw floor(z * m / 2^64),
  and a partial Fisher-Yates shuffle of the candidate list.
  The paper prints no sample layout; the stream is pinned to SplitMix64's
  published outputs and the selection to vectors worked by hand from them
  (tests/golden/random_blocks_seed0.txt), besides its invariants and statistics.
  seed < 2^24 and h, j < 2^20 (the key's field widths).
* Padding: keys whose key_padding_mask is 0 get score -inf before the softmax;
  the attention graph itself does not depend on the mask.
* lse is the natural log of the sum of exp(scaled, masked scores).

* Backward pass (the paper trains through this op, Sec. 4 "Pretraining and MLM",
  App. E.1, but prints no gradient formulas): the textbook derivatives of
  Eq. (AT) under the same mask, written out in `attend_bwd`.  Padded QUERY rows
  receive no gradient and give none (the library returns out = 0 for them).

Everything is fp64.  Nothing here is blocked, fused or reordered.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

MASK64 = (1 << 64) - 1
ITC = 0
ETC = 1


@dataclass(frozen=True)
class Graph:
    """Parameters of one BigBird attention graph (App. D; w, g, r in blocks)."""
    N: int
    b: int
    w: int
    g: int
    r: int
    seed: int
    H: int
    mode: int = ITC

    def __post_init__(self):
        if self.N <= 0 or self.b <= 0 or self.N % self.b:
            raise ValueError("N must be a positive multiple of b")
        if self.w < 1 or self.w % 2 == 0:
            raise ValueError("w must be odd and >= 1")
        if self.g < 0 or self.r < 0 or self.H < 1 or self.g > self.N // self.b:
            raise ValueError("bad g, r or H")
        if self.mode not in (ITC, ETC):
            raise ValueError("mode")
        # field widths of the stream key (seed << 40) ^ (h << 20) ^ j: 24 bits of seed, 20 of head, 20 of block
        if not (0 <= self.seed < (1 << 24)) or self.H > (1 << 20) or self.N // self.b > (1 << 20):
            raise ValueError("seed must be below 2^24, heads and blocks at most 2^20")

    @property
    def nb(self) -> int:
        return self.N // self.b


# --------------------------------------------------------------------------
# The random stream (not from the paper; see the header).
# --------------------------------------------------------------------------
def splitmix64_next(state: int) -> Tuple[int, int]:
    """One SplitMix64 step: returns (new_state, output)."""
    state = (state + 0x9E3779B97F4A7C15) & MASK64
    z = state
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & MASK64
    z = z ^ (z >> 31)
    return state, z


def stream_key(seed: int, h: int, j: int) -> int:
    return (((seed << 40) & MASK64) ^ (h << 20) ^ j) & MASK64


def global_blocks(gr: Graph) -> List[int]:
    """Sec. 2 (ITC / ETC definitions of G), at block granularity (App. D item 3)."""
    if gr.mode == ETC:
        return list(range(gr.g))
    first = (gr.g + 1) // 2
    last = gr.g // 2
    return sorted(set(range(first)) | set(range(gr.nb - last, gr.nb)))


def window_blocks(gr: Graph, j: int) -> List[int]:
    """App. D item 2: key blocks j-(w-1)/2 .. j+(w-1)/2, clipped to the sequence."""
    hw = (gr.w - 1) // 2
    return [c for c in range(j - hw, j + hw + 1) if 0 <= c < gr.nb]


def random_blocks(gr: Graph, h: int, j: int) -> List[int]:
    """App. D item 1: the r random key blocks of query block j in head h."""
    G = set(global_blocks(gr))
    if j in G or gr.r == 0:
        return []
    W = set(window_blocks(gr, j))
    cand = [c for c in range(gr.nb) if c not in G and c not in W]
    m = len(cand)
    take = min(gr.r, m)
    state = stream_key(gr.seed, h, j)
    for t in range(take):
        state, z = splitmix64_next(state)
        p = t + ((z * (m - t)) >> 64)
        cand[t], cand[p] = cand[p], cand[t]
    return sorted(cand[:take])


# --------------------------------------------------------------------------
# The adjacency matrix A (Sec. 2), built token by token.
# --------------------------------------------------------------------------
def mask_rows(gr: Graph, h: int, rows: Sequence[int]) -> np.ndarray:
    """A[h][rows, :] as bool[len(rows), N]: A(i, k) = 1 iff query i attends key k.

    With I = floor(i/b) and C = floor(k/b): global row (I in G) or global column
    (C in G) or window (|I - C| <= (w-1)/2) or C in the random set of (h, I).
    """
    rows = np.asarray(rows, dtype=np.int64)
    hw = (gr.w - 1) // 2
    isG = np.zeros(gr.nb, dtype=bool)
    isG[global_blocks(gr)] = True
    I = rows // gr.b
    C = np.arange(gr.N, dtype=np.int64) // gr.b
    A = np.zeros((len(rows), gr.N), dtype=bool)
    A |= isG[I][:, None]
    A |= isG[C][None, :]
    A |= np.abs(I[:, None] - C[None, :]) <= hw
    rnd = np.zeros((gr.nb, gr.nb), dtype=bool)
    for Ib in np.unique(I):
        rnd[Ib, random_blocks(gr, h, int(Ib))] = True
    A |= rnd[I[:, None], C[None, :]]
    return A


def build_mask(gr: Graph, h: int) -> np.ndarray:
    """The full N x N adjacency matrix of head h."""
    return mask_rows(gr, h, np.arange(gr.N))


def layout_from_mask(gr: Graph) -> Tuple[np.ndarray, np.ndarray]:
    """Key-block lists read off the token-level mask, as CSR over (head, query block).

    Row (h, I) lists, ascending, the key blocks C with A[h](I*b, C*b) = 1.
    Returns (row_ptr int32[H*nb + 1], col_idx int32[nnz]).
    """
    row_ptr = [0]
    cols: List[int] = []
    first_tokens = np.arange(gr.nb, dtype=np.int64) * gr.b
    for h in range(gr.H):
        A = mask_rows(gr, h, first_tokens)[:, first_tokens]
        for I in range(gr.nb):
            cs = np.nonzero(A[I])[0]
            cols.extend(int(c) for c in cs)
            row_ptr.append(len(cols))
    return np.asarray(row_ptr, dtype=np.int32), np.asarray(cols, dtype=np.int32)


# --------------------------------------------------------------------------
# Eq. (AT): masked softmax attention, fp64.
# --------------------------------------------------------------------------
def attend(q_rows: np.ndarray, k: np.ndarray, v: np.ndarray, A_rows: np.ndarray,
           key_valid: Optional[np.ndarray], scale: float) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. (AT) for a set of query rows of one (batch, head).

    q_rows [R, D], k [N, D], v [N, D], A_rows bool[R, N], key_valid bool[N] or None.
    Returns out fp64[R, D] and lse fp64[R].  A row with no attended valid key
    gets out = 0 and lse = -inf.
    """
    q_rows = np.asarray(q_rows, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    S = scale * (q_rows @ k.T)
    keep = A_rows if key_valid is None else (A_rows & np.asarray(key_valid, dtype=bool)[None, :])
    S = np.where(keep, S, -np.inf)
    m = S.max(axis=1)
    safe_m = np.where(np.isfinite(m), m, 0.0)
    E = np.exp(S - safe_m[:, None])
    l = E.sum(axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        lse = np.where(l > 0, safe_m + np.log(l), -np.inf)
        P = np.where(l[:, None] > 0, E / l[:, None], 0.0)
    return P @ v, lse


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, gr: Graph,
              key_padding_mask: Optional[np.ndarray], scale: float,
              slices: Optional[Sequence[Tuple[int, int]]] = None,
              rows: Optional[Sequence[int]] = None) -> Dict[Tuple[int, int], Tuple[np.ndarray, np.ndarray]]:
    """BigBird attention for [B, H, N, D] inputs.

    Returns {(batch, head): (out fp64[R, D], lse fp64[R])} for the requested
    (batch, head) slices (all by default) and query rows (all by default).
    """
    B, H, N, D = q.shape
    assert H == gr.H and N == gr.N
    if slices is None:
        slices = [(bi, h) for bi in range(B) for h in range(H)]
    rws = np.arange(N) if rows is None else np.asarray(rows, dtype=np.int64)
    res = {}
    masks: Dict[int, np.ndarray] = {}
    for (bi, h) in slices:
        if h not in masks:
            masks = {h: mask_rows(gr, h, rws)}      # keep only one head's mask alive
        kv = None if key_padding_mask is None else (np.asarray(key_padding_mask[bi]) != 0)
        res[(bi, h)] = attend(np.asarray(q[bi, h], dtype=np.float64)[rws], k[bi, h], v[bi, h],
                              masks[h], kv, scale)
    return res


# --------------------------------------------------------------------------
# Gradients of Eq. (AT) (the paper trains through the op; it prints no formulas).
# --------------------------------------------------------------------------
def attend_bwd(q_rows: np.ndarray, k: np.ndarray, v: np.ndarray, A_rows: np.ndarray,
               key_valid: Optional[np.ndarray], scale: float, dout_rows: np.ndarray,
               row_valid: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Gradients of sum(out * dout) for a set of query rows of one (batch, head).

    With S = scale q k^T restricted to the attended valid keys, P = softmax(S) and
    out = P v:  dv = P^T dout,  dP = dout v^T,  dS = P o (dP - rowsum(dout o out)),
    dq = scale dS k,  dk = scale dS^T q.  Rows with row_valid == False (padded
    queries) and rows without any attended valid key contribute nothing and get
    dq = 0.  Returns (dq fp64[R, D], dk fp64[N, D], dv fp64[N, D]); dk and dv
    hold the contribution of these rows only.
    """
    q_rows = np.asarray(q_rows, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout_rows = np.asarray(dout_rows, dtype=np.float64)
    S = scale * (q_rows @ k.T)
    keep = A_rows if key_valid is None else (A_rows & np.asarray(key_valid, dtype=bool)[None, :])
    if row_valid is not None:
        keep = keep & np.asarray(row_valid, dtype=bool)[:, None]
    S = np.where(keep, S, -np.inf)
    m = S.max(axis=1)
    safe_m = np.where(np.isfinite(m), m, 0.0)
    E = np.exp(S - safe_m[:, None])
    l = E.sum(axis=1)
    with np.errstate(divide="ignore", invalid="ignore"):
        P = np.where(l[:, None] > 0, E / l[:, None], 0.0)
    out = P @ v
    dv = P.T @ dout_rows
    dP = dout_rows @ v.T
    delta = (dout_rows * out).sum(axis=1)
    dS = P * (dP - delta[:, None])
    dq = scale * (dS @ k)
    dk = scale * (dS.T @ q_rows)
    return dq, dk, dv


def attention_bwd(q: np.ndarray, k: np.ndarray, v: np.ndarray, dout: np.ndarray, gr: Graph,
                  key_padding_mask: Optional[np.ndarray], scale: float,
                  slices: Optional[Sequence[Tuple[int, int]]] = None
                  ) -> Dict[Tuple[int, int], Tuple[np.ndarray, np.ndarray, np.ndarray]]:
    """BigBird attention gradients for [B, H, N, D] inputs: {(batch, head): (dq, dk, dv)} in fp64."""
    B, H, N, D = q.shape
    assert H == gr.H and N == gr.N
    if slices is None:
        slices = [(bi, h) for bi in range(B) for h in range(H)]
    res = {}
    masks: Dict[int, np.ndarray] = {}
    for (bi, h) in slices:
        if h not in masks:
            masks = {h: build_mask(gr, h)}
        kv = None if key_padding_mask is None else (np.asarray(key_padding_mask[bi]) != 0)
        res[(bi, h)] = attend_bwd(q[bi, h], k[bi, h], v[bi, h], masks[h], kv, scale, dout[bi, h], row_valid=kv)
    return res
