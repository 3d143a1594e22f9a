"""CPU oracle for the Bi-Mask per-layer sparse training step.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of the
method that the CUDA path is checked against.  Only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may import it; the product path
never does.  It shares no code with the CUDA path and imports nothing from the
package.

Notation follows the paper: W is I x J (output rows x input dim), B is the
forward N:M mask (N:M along each row, Eq. 2 / Eq. 4), B-bar the backward mask
(N:M along each column of the row-permuted matrix, Eq. 7 / Eq. 11), `perm` the
row permutation vector of Eq. 10 (gather: Wp[k, :] = W[perm[k], :], 0-based).

All arrays are numpy.  Floating-point products are done in float64.  Integer
results (mask bits, packed indices, counts, the chosen permutation) are exact.

Readings of points the paper leaves open:
  * blocks are the aligned, disjoint index ranges [g*M, (g+1)*M), 0-based;
  * "Top(., N)" of Eq. 4 / Eq. 11 is applied as a rank: an element is kept when
    fewer than N elements of its block beat it, where an element q beats m if
    its magnitude is larger, or equal with q < m.  With distinct magnitudes
    this is Eq. 4 / Eq. 11 verbatim; with ties it keeps exactly N (Eq. 2);
  * magnitudes are compared on the fp32 weights through the integer key
    bits(w) & 0x7fffffff (monotone in |w|, -0 == +0);
  * in the backward mask only positions with a forward bit of 1 are ranked, so
    B-bar is always a subset of B[perm] (the paper's second rationale for
    Eq. 9), also when a kept weight is exactly zero;
  * an "eligible" column block (the quantity the permutation search counts,
    Alg. 1) has at most N forward-mask bits among its M rows;
  * ties between candidate permutations go to the lowest candidate index;
  * the weight gradient is the dense straight-through one, dW = dY^T X;
  * the optimizer update (`sgd_update`) is float32 in a fixed operation order,
    because the updated weights decide the next mask; the permutation is the
    identity before the first search; interval q = t // Delta T draws its
    candidates from seed + q;
  * the ablation's other backward-mask criteria (`backward_mask_criterion`):
    "multinomial" is N draws without replacement proportional to |w| by
    inverse CDF in float32; "random" ranks hashed per-weight keys.

Parity unpinned: the pseudo-random candidate generator (`candidates`).  The
paper only says the K candidates are random; the generator below is this
build's contract (its mixing function is pinned to the published SplitMix64
test vector, the rest by permutation validity, a uniformity test and a
three-candidate vector computed independently from the written definition).
"""
from __future__ import annotations

import numpy as np

MASK64 = (1 << 64) - 1


# --------------------------------------------------------------------------
# helpers: magnitude key, bf16 rounding
# --------------------------------------------------------------------------
def magnitude_key(W: np.ndarray) -> np.ndarray:
    """Integer magnitude of fp32 values: the bit pattern with the sign cleared."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    return (W.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bfloat16 (round to nearest, ties to even); returns uint16 bit patterns.

    NaN becomes a quiet NaN with the sign kept; infinities are kept."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    rounded = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    is_nan = (u & np.uint64(0x7FFFFFFF)) > np.uint64(0x7F800000)
    nan_bits = (u >> np.uint64(16)) | np.uint64(0x0040)
    return np.where(is_nan, nan_bits, rounded).astype(np.uint16)


def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bfloat16 bit patterns, as float64."""
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def bf16_round(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 -> float64 (the value the tensor core sees)."""
    return bf16_to_f64(bf16_bits(x))


# --------------------------------------------------------------------------
# Eq. 4: forward mask
# --------------------------------------------------------------------------
def _rank_keep(key: np.ndarray, valid: np.ndarray, N: int) -> np.ndarray:
    """key, valid: (..., M).  Keep element m iff it is valid and fewer than N valid
    elements of its block beat it (larger key, or equal key at a lower position)."""
    M = key.shape[-1]
    keep = np.zeros(key.shape, dtype=bool)
    for m in range(M):
        beaten_by = np.zeros(key.shape[:-1], dtype=np.int64)
        for q in range(M):
            if q == m:
                continue
            if q < m:
                beats = key[..., q] >= key[..., m]
            else:
                beats = key[..., q] > key[..., m]
            beaten_by += (beats & valid[..., q]).astype(np.int64)
        keep[..., m] = valid[..., m] & (beaten_by < N)
    return keep


def forward_mask(W: np.ndarray, N: int, M: int) -> np.ndarray:
    """Eq. 4 (constraint Eq. 2): B[i, gM:(g+1)M] keeps the N largest |W| of the block.

    Returns a bool array I x J with exactly N ones in every aligned row block."""
    I, J = W.shape
    assert J % M == 0 and 1 <= N <= M
    key = magnitude_key(W).reshape(I, J // M, M)
    keep = _rank_keep(key, np.ones_like(key, dtype=bool), N)
    return keep.reshape(I, J)


# --------------------------------------------------------------------------
# Alg. 1 (permutation step): candidates, eligible-block count, pick
# --------------------------------------------------------------------------
def _mix64(z: int) -> int:
    z &= MASK64
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & MASK64
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & MASK64
    z ^= z >> 31
    return z


def _mix64_np(z: np.ndarray) -> np.ndarray:
    z = z.astype(np.uint64)
    z ^= z >> np.uint64(30)
    z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27)
    z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def candidates(seed: int, P: int, I: int) -> np.ndarray:
    """P pseudo-random permutations of {0..I-1} (the K random candidates of the permutation step of Alg. 1).

    Candidate c sorts the rows by a hashed key: row i gets
        h = mix64(mix64(seed + 0x9E3779B97F4A7C15 * (c + 1)) ^ i)
    and the sort key (h with its low 24 bits replaced by i), so keys are distinct
    and the result does not depend on the sorting algorithm.  Requires I < 2**24."""
    assert 0 < I < (1 << 24) and P >= 1
    out = np.empty((P, I), dtype=np.int32)
    rows = np.arange(I, dtype=np.uint64)
    with np.errstate(over="ignore"):
        for c in range(P):
            stream = _mix64((seed + 0x9E3779B97F4A7C15 * (c + 1)) & MASK64)
            h = _mix64_np(np.uint64(stream) ^ rows)
            v = (h & ~np.uint64(0xFFFFFF)) | rows
            v.sort()
            out[c] = (v & np.uint64(0xFFFFFF)).astype(np.int32)
    return out


def eligible_blocks(B: np.ndarray, perm: np.ndarray, N: int, M: int) -> int:
    """Number of (row block k, column l) pairs of B[perm, :] that already satisfy N:M,
    i.e. hold at most N ones among rows kM..kM+M-1 (the paper's "eligible N:M blocks")."""
    I, J = B.shape
    assert I % M == 0
    Bp = B[np.asarray(perm, dtype=np.int64), :]
    pop = Bp.reshape(I // M, M, J).sum(axis=1)
    return int((pop <= N).sum())


def perm_search(B: np.ndarray, cands: np.ndarray, N: int, M: int):
    """Alg. 1, permutation step: score every candidate, pick the one with the most
    eligible blocks (lowest index on ties).  Returns (best_idx, best_perm, counts)."""
    counts = np.array([eligible_blocks(B, c, N, M) for c in cands], dtype=np.int64)
    best = int(np.argmax(counts))          # argmax returns the first maximum
    return best, np.array(cands[best], dtype=np.int32), counts


# --------------------------------------------------------------------------
# Eq. 11 (Eq. 9 when perm is the identity): backward mask
# --------------------------------------------------------------------------
def backward_mask(W: np.ndarray, B: np.ndarray, perm: np.ndarray, N: int, M: int) -> np.ndarray:
    """Eq. 11: on the row-permuted masked weights (B*W)[perm, :], every aligned block of M
    rows of every column keeps its N largest magnitudes among the entries whose forward
    bit is set.  Returns B-bar (bool, I x J) in PERMUTED row order (row k <-> W row perm[k])."""
    I, J = W.shape
    assert I % M == 0 and 1 <= N <= M
    p = np.asarray(perm, dtype=np.int64)
    key = magnitude_key(W)[p, :].reshape(I // M, M, J).transpose(0, 2, 1)   # (blocks, J, M)
    valid = B[p, :].reshape(I // M, M, J).transpose(0, 2, 1)
    keep = _rank_keep(key, valid, N)
    return keep.transpose(0, 2, 1).reshape(I, J)


def unpermute_rows(Bbar_p: np.ndarray, perm: np.ndarray) -> np.ndarray:
    """M_b[perm[k], :] = B-bar[k, :]  (backward mask in the original row order)."""
    out = np.zeros_like(Bbar_p)
    out[np.asarray(perm, dtype=np.int64), :] = Bbar_p
    return out


# --------------------------------------------------------------------------
# 2:4 operand format (not in the paper; defined by this build's interface)
# --------------------------------------------------------------------------
def pack_bits(mask: np.ndarray) -> np.ndarray:
    """bool R x C (C % 32 == 0) -> uint32 R x C/32, bit (c % 32) of word c // 32."""
    R, C = mask.shape
    assert C % 32 == 0
    m = mask.reshape(R, C // 32, 32).astype(np.uint64)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    return (m * weights).sum(axis=2).astype(np.uint32)


def unpack_bits(words: np.ndarray, C: int) -> np.ndarray:
    R = words.shape[0]
    w = words.astype(np.uint64)[:, :, None] >> np.arange(32, dtype=np.uint64)
    return (w & np.uint64(1)).astype(bool).reshape(R, -1)[:, :C]


def pack_2to4(A: np.ndarray, keep: np.ndarray):
    """Compress a matrix whose kept entries number at most 2 per aligned group of 4 along
    the rows into the 2:4 tensor-core operand: two bf16 values and one 4-bit index code
    per group.

    A: fp32 R x C, keep: bool R x C.  Returns (vals uint16 R x C/2, meta uint32 R x C/32).
    Per group: S = kept positions ascending.  Fewer than 2 kept: pad with the lowest
    positions not in S and sort.  Code = idx0 | idx1 << 2; slot s holds bf16(A[idx_s]) if
    idx_s is kept, else +0.  Code g of a row sits in bits [4 (g % 8), +4) of word g // 8."""
    R, C = A.shape
    assert C % 32 == 0
    G = C // 4
    keep4 = keep.reshape(R, G, 4)
    assert int(keep4.sum(axis=2).max(initial=0)) <= 2
    abits = bf16_bits(A).reshape(R, G, 4)
    vals = np.zeros((R, G, 2), dtype=np.uint16)
    code = np.zeros((R, G), dtype=np.uint32)
    for r in range(R):
        for g in range(G):
            S = [m for m in range(4) if keep4[r, g, m]]
            idx = list(S)
            m = 0
            while len(idx) < 2:
                if m not in idx:
                    idx.append(m)
                m += 1
            idx.sort()
            code[r, g] = idx[0] | (idx[1] << 2)
            for s in range(2):
                vals[r, g, s] = abits[r, g, idx[s]] if idx[s] in S else 0
    shifts = (4 * (np.arange(G) % 8)).astype(np.uint32)
    meta = (code << shifts).reshape(R, G // 8, 8).sum(axis=2).astype(np.uint32)
    return vals.reshape(R, C // 2), meta


def pack_2to4_fast(A: np.ndarray, keep: np.ndarray):
    """Same result as pack_2to4, vectorised over groups (used at sizes where the
    per-group Python loop would take minutes).  Checked against pack_2to4 in the tests."""
    R, C = A.shape
    assert C % 32 == 0
    G = C // 4
    keep4 = keep.reshape(R, G, 4)
    cnt = keep4.sum(axis=2)
    assert int(cnt.max(initial=0)) <= 2
    abits = bf16_bits(A).reshape(R, G, 4)
    pos = np.arange(4)
    # first and last kept position of each group
    first = np.where(keep4, pos, 9).min(axis=2)
    last = np.where(keep4, pos, -1).max(axis=2)
    idx0 = np.zeros((R, G), dtype=np.int64)
    idx1 = np.ones((R, G), dtype=np.int64)
    two = cnt == 2
    idx0[two] = first[two]
    idx1[two] = last[two]
    one = cnt == 1
    p = first[one]
    idx0[one] = 0
    idx1[one] = np.where(p <= 1, 1, p)
    code = (idx0 | (idx1 << 2)).astype(np.uint32)
    take0 = np.take_along_axis(abits, idx0[..., None], axis=2)[..., 0]
    take1 = np.take_along_axis(abits, idx1[..., None], axis=2)[..., 0]
    kept0 = np.take_along_axis(keep4, idx0[..., None], axis=2)[..., 0]
    kept1 = np.take_along_axis(keep4, idx1[..., None], axis=2)[..., 0]
    vals = np.stack([np.where(kept0, take0, 0), np.where(kept1, take1, 0)], axis=2).astype(np.uint16)
    shifts = (4 * (np.arange(G) % 8)).astype(np.uint32)
    meta = (code << shifts).reshape(R, G // 8, 8).sum(axis=2).astype(np.uint32)
    return vals.reshape(R, C // 2), meta


def unpack_2to4(vals: np.ndarray, meta: np.ndarray) -> np.ndarray:
    """Expand a packed 2:4 operand back to a dense float64 R x C matrix."""
    R, half = vals.shape
    G = half // 2
    v = bf16_to_f64(vals).reshape(R, G, 2)
    out = np.zeros((R, G, 4), dtype=np.float64)
    for r in range(R):
        for g in range(G):
            c = (int(meta[r, g // 8]) >> (4 * (g % 8))) & 0xF
            # a slot holding +0 adds nothing, so a padded slot never disturbs a kept one
            out[r, g, c & 3] += v[r, g, 0]
            out[r, g, (c >> 2) & 3] += v[r, g, 1]
    return out.reshape(R, 4 * G)


def dense_operand(A: np.ndarray, keep: np.ndarray) -> np.ndarray:
    """Masked operand for patterns the 2:4 tensor-core format cannot hold (more than two survivors
    in some aligned group of four, e.g. 4:8): bf16 bit patterns of A where `keep`, +0 elsewhere."""
    return np.where(keep, bf16_bits(A), np.uint16(0)).astype(np.uint16)


def dense_backward_operand(W: np.ndarray, Bbar_p: np.ndarray, perm: np.ndarray) -> np.ndarray:
    """(B-bar * W[perm, :])^T as a dense bf16 J x I matrix (reduction index = permuted rows)."""
    Wp = np.ascontiguousarray(W[np.asarray(perm, dtype=np.int64), :], dtype=np.float32)
    return dense_operand(np.ascontiguousarray(Wp.T), np.ascontiguousarray(Bbar_p.T))


def forward_operand(W: np.ndarray, B: np.ndarray):
    """Packed forward operand A_f = B*W (I x J, 2:4 along J): (maskbits, vals, meta)."""
    vals, meta = pack_2to4_fast(W, B)
    return pack_bits(B), vals, meta


def backward_operand(W: np.ndarray, Bbar_p: np.ndarray, perm: np.ndarray):
    """Packed backward operand A' = (B-bar * W[perm, :])^T  (J x I, 2:4 along the permuted
    rows of W, which is the reduction dim of Eq. 10): (maskbits of B-bar, vals, meta)."""
    Wp = np.ascontiguousarray(W[np.asarray(perm, dtype=np.int64), :], dtype=np.float32)
    vals, meta = pack_2to4_fast(np.ascontiguousarray(Wp.T), np.ascontiguousarray(Bbar_p.T))
    return pack_bits(Bbar_p), vals, meta


# --------------------------------------------------------------------------
# Eq. 3, Eq. 8 / Eq. 10, STE weight gradient
# --------------------------------------------------------------------------
def spmm_fwd(X_bits: np.ndarray, W: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Eq. 3 in the row-major activation layout: Y[t, i] = sum_j X[t, j] (B*W)[i, j],
    on bf16-rounded W and bf16 X, accumulated in float64."""
    Wf = bf16_round(W) * B
    return bf16_to_f64(X_bits) @ Wf.T


def spmm_dgrad(dY_bits: np.ndarray, W: np.ndarray, Mb: np.ndarray) -> np.ndarray:
    """Eq. 8: dX[t, j] = sum_i dY[t, i] (M_b*W)[i, j], with M_b the backward mask in the
    original row order (the unpermuted form, which Eq. 10 says equals the permuted one)."""
    Wb = bf16_round(W) * Mb
    return bf16_to_f64(dY_bits) @ Wb


def spmm_dgrad_permuted(dY_bits: np.ndarray, W: np.ndarray, Bbar_p: np.ndarray, perm: np.ndarray) -> np.ndarray:
    """Eq. 10 as printed: (B-bar * W[perm, :])^T applied to dY[:, perm]."""
    p = np.asarray(perm, dtype=np.int64)
    Wp = bf16_round(W)[p, :] * Bbar_p
    return bf16_to_f64(dY_bits)[:, p] @ Wp


def dense_dgrad(dY_bits: np.ndarray, W: np.ndarray, B: np.ndarray) -> np.ndarray:
    """Eq. 5: the exact input gradient through the forward mask (what Bi-Mask approximates)."""
    return bf16_to_f64(dY_bits) @ (bf16_round(W) * B)


def wgrad(dY_bits: np.ndarray, X_bits: np.ndarray) -> np.ndarray:
    """Straight-through weight gradient: dW[i, j] = sum_t dY[t, i] X[t, j] (dense, unmasked)."""
    return bf16_to_f64(dY_bits).T @ bf16_to_f64(X_bits)


# --------------------------------------------------------------------------
# Alg. 1 body for one layer
# --------------------------------------------------------------------------
def layer_step(W, X_bits, dY_bits, N, M, P, seed, do_search=True, perm=None, cands=None,
               with_gemms=True):
    """One iteration of Alg. 1 for one layer, minus the optimizer update.

    Returns a dict with B, the packed forward operand, the candidates' counts, the chosen
    permutation, B-bar (permuted order), M_b, the packed backward operand and, when
    with_gemms, Y, dX and dW (float64)."""
    I, J = W.shape
    out = {}
    B = forward_mask(W, N, M)
    out["B"] = B
    packable = (M % 4 == 0 and N <= 2)  # at most two survivors in every aligned group of four: fits the 2:4 operand
    if packable:
        out["maskbits_f"], out["vals_f"], out["meta_f"] = forward_operand(W, B)
    if do_search:
        if cands is None:
            cands = candidates(seed, P, I)
        best, perm, counts = perm_search(B, cands, N, M)
        out["best_idx"], out["counts"] = best, counts
    else:
        perm = np.arange(I, dtype=np.int32) if perm is None else np.asarray(perm, dtype=np.int32)
    out["perm"] = perm
    Bbar_p = backward_mask(W, B, perm, N, M)
    out["Bbar_p"] = Bbar_p
    out["M_b"] = unpermute_rows(Bbar_p, perm)
    if packable:
        out["maskbits_b"], out["vals_b"], out["meta_b"] = backward_operand(W, Bbar_p, perm)
    if with_gemms:
        out["Y"] = spmm_fwd(X_bits, W, B)
        out["dX"] = spmm_dgrad(dY_bits, W, out["M_b"])
        out["dW"] = wgrad(dY_bits, X_bits)
    return out


# ---------------------------------------------------------------------------------------
# Algorithm 1 as a loop: the Delta-T schedule of the search and the optimizer update
# ---------------------------------------------------------------------------------------

def sgd_update(W, dW, mom, lr, momentum, weight_decay):
    """The optimizer update that ends the loop body of Algorithm 1 (Sec. 4.1 trains with SGD,
    momentum and weight decay).  The straight-through estimator hands the gradient of B.W to the dense
    weights unchanged (Sec. 3.1), so the update runs on all of W:

        g = dW + weight_decay * W ;  mom = momentum * mom + g ;  W = W - lr * mom

    The updated weights decide the next forward mask (an integer result), so the arithmetic is pinned
    to the precision of the stored weights: float32, every product and sum rounded once, in exactly
    the order written above (no fused multiply-add).  Returns (W_new, mom_new), float32."""
    f = np.float32
    W = np.asarray(W, dtype=f)
    dW = np.asarray(dW, dtype=f)
    mom = np.asarray(mom, dtype=f)
    g = dW + f(weight_decay) * W
    mom_new = f(momentum) * mom + g
    W_new = W - f(lr) * mom_new
    return W_new.astype(f), mom_new.astype(f)


def interval_seed(seed, t, delta_t):
    """Seed of the candidates drawn at iteration t: each interval draws fresh candidates
    (Sec. 3.2: K new random permutations every Delta T iterations); interval number = t // delta_t."""
    return (int(seed) + int(t) // int(delta_t)) & MASK64


def train_steps(W0, X_bits, dY_bits, N, M, P, seed, delta_t, iters, lr, momentum, weight_decay,
                with_gemms=True):
    """Algorithm 1 for one layer: for t = 1 .. iters: forward mask (Eq. 4), forward product (Eq. 3),
    if t % delta_t == 0 a new search, backward mask (Eq. 11), input gradient (Eq. 10), dense weight
    gradient, SGD update.  Before the first search the permutation is the identity.  X_bits / dY_bits
    are lists with one entry per iteration (or a single array used every iteration).

    Returns (history, W_final, mom_final, sparse_final) where history[t-1] is layer_step's dict for
    iteration t plus 'W' (the weights that iteration saw) and 'searched'; sparse_final = B . W for the
    mask of the final weights (the algorithm's return value)."""
    W = np.asarray(W0, dtype=np.float32).copy()
    mom = np.zeros_like(W)
    perm = np.arange(W.shape[0], dtype=np.int32)
    history = []
    for t in range(1, iters + 1):
        Xb = X_bits[t - 1] if isinstance(X_bits, (list, tuple)) else X_bits
        dYb = dY_bits[t - 1] if isinstance(dY_bits, (list, tuple)) else dY_bits
        searched = (t % delta_t == 0)
        out = layer_step(W, Xb, dYb, N, M, P, interval_seed(seed, t, delta_t), do_search=searched,
                         perm=perm, with_gemms=with_gemms)
        perm = out["perm"]
        out["W"] = W.copy()
        out["searched"] = searched
        dW = out["dW"] if with_gemms else wgrad(dYb, Xb)
        W, mom = sgd_update(W, np.asarray(dW, dtype=np.float64).astype(np.float32), mom, lr, momentum,
                            weight_decay)
        history.append(out)
    B = forward_mask(W, N, M)
    return history, W, mom, np.where(B, W, np.float32(0))


# ---------------------------------------------------------------------------------------
# Other criteria for the backward mask (the ablation on binarization criteria, Sec. 4.4 / Table 8)
# ---------------------------------------------------------------------------------------
CRIT_WEIGHT, CRIT_SCORE, CRIT_MULTINOMIAL, CRIT_RANDOM = 0, 1, 2, 3
_GAMMA = 0x9E3779B97F4A7C15


def random_keys(seed: int, I: int, J: int) -> np.ndarray:
    """31-bit pseudo-random key of every weight (i, j), a function of (seed, i*J + j) only:
    mix64(mix64(seed) + i*J + j) >> 33."""
    e = np.arange(I * J, dtype=np.uint64).reshape(I, J)
    with np.errstate(over="ignore"):
        return (_mix64_np(np.uint64(_mix64(seed)) + e) >> np.uint64(33)).astype(np.int64)


def _uniform24(seed: int, draw: int, index: np.ndarray) -> np.ndarray:
    """Uniform in [0, 1) with 24 bits, exactly representable in float32: a function of
    (seed, draw number, block index)."""
    with np.errstate(over="ignore"):
        h = _mix64_np(np.uint64(_mix64((seed + _GAMMA * (draw + 1)) & MASK64)) ^ index.astype(np.uint64))
    return ((h >> np.uint64(40)).astype(np.float32) * np.float32(2.0 ** -24)).astype(np.float32)


def backward_mask_criterion(W, B, perm, N, M, criterion, S=None, seed=0):
    """Backward mask with the N survivors of a column block chosen by another criterion than the
    weight magnitude (the paper's ablation compares: weight magnitude -- Eq. 11, its choice --,
    gradient magnitude, multinomial sampling by magnitude, and random).  As in Eq. 11 only entries
    whose forward bit is set compete, blocks are M consecutive rows of the permuted matrix, and a
    block with at most N competitors keeps them all.  Returns B-bar in permuted row order.

      CRIT_WEIGHT       Eq. 11 (backward_mask).
      CRIT_SCORE        rank by |S[perm]| instead of |W[perm]| (S = the weight gradient gives the
                        gradient-magnitude variant); ties to the lower row of the block.
      CRIT_RANDOM       rank by random_keys(seed): a uniformly random N-subset of the competitors.
      CRIT_MULTINOMIAL  N draws without replacement, each proportional to |w| among the remaining
                        competitors: with a = |w| in float32 and u = _uniform24(seed, draw, block),
                        x = u * (a_0 + a_1 + ...) summed in row order, the draw takes the first
                        remaining competitor whose running sum exceeds x; if none does (all zero,
                        non-finite, or u*total rounded up to the total) the lowest remaining one.
                        Every product and sum is float32, rounded once, so the draw is reproducible
                        bit for bit."""
    I, J = W.shape
    assert I % M == 0 and 1 <= N <= M
    p = np.asarray(perm, dtype=np.int64)
    nb = I // M
    valid = B[p, :].reshape(nb, M, J).transpose(0, 2, 1)                    # (blocks, J, M)
    if criterion == CRIT_WEIGHT:
        return backward_mask(W, B, perm, N, M)
    if criterion in (CRIT_SCORE, CRIT_RANDOM):
        full = magnitude_key(S) if criterion == CRIT_SCORE else random_keys(seed, I, J)
        key = full[p, :].reshape(nb, M, J).transpose(0, 2, 1)
        return _rank_keep(key, valid, N).transpose(0, 2, 1).reshape(I, J)
    assert criterion == CRIT_MULTINOMIAL
    f = np.float32
    a = np.abs(np.asarray(W, dtype=f))[p, :].reshape(nb, M, J).transpose(0, 2, 1)
    remaining = valid.copy()
    keep = np.zeros_like(valid)
    many = valid.sum(axis=2) > N                                             # blocks that must choose
    block_index = (np.arange(nb, dtype=np.uint64)[:, None] * np.uint64(J) + np.arange(J, dtype=np.uint64)[None, :])
    for d in range(N):
        u = _uniform24(seed, d, block_index)
        total = np.zeros((nb, J), dtype=f)
        for m in range(M):
            total = np.where(remaining[..., m], total + a[..., m], total).astype(f)
        with np.errstate(invalid="ignore", over="ignore"):
            x = (u * total).astype(f)
        chosen = np.full((nb, J), -1, dtype=np.int64)
        cum = np.zeros((nb, J), dtype=f)
        for m in range(M):
            cum = np.where(remaining[..., m], cum + a[..., m], cum).astype(f)
            with np.errstate(invalid="ignore"):
                hit = remaining[..., m] & (cum > x) & (chosen < 0)
            chosen = np.where(hit, m, chosen)
        lowest = np.argmax(remaining, axis=2)                                # first remaining competitor
        chosen = np.where(chosen < 0, lowest, chosen)
        sel = np.zeros_like(valid)
        np.put_along_axis(sel, chosen[..., None], True, axis=2)
        sel &= remaining                                                     # (no competitor left: nothing)
        keep |= sel
        remaining &= ~sel
    keep = np.where(many[..., None], keep, valid)
    return keep.transpose(0, 2, 1).reshape(I, J)


# ---------------------------------------------------------------------------------------
# The same layer step when the layer is a 3x3 convolution (stride 1, zero padding 1) on NHWC
# activations: "W" of the paper is the I x J matrix view of the filter, J = 9*C, column
# j = (kh*3 + kw)*C + c (the paper does not state the flatten order; this one keeps the channel
# index contiguous, as in the NHWC activations).
# ---------------------------------------------------------------------------------------
def _pad_hw(a):
    return np.pad(a, ((0, 0), (1, 1), (1, 1), (0, 0)))


def conv_out_size(n: int, stride: int) -> int:
    """Output extent of a 3-tap window with padding 1: floor((n + 2 - 3) / stride) + 1."""
    return (n - 1) // stride + 1


def conv_fwd(x_bits, W, B, stride=1):
    """y[n, ho, wo, i] = sum_{kh, kw, c} x[n, ho*s+kh-1, wo*s+kw-1, c] * (B.W)[i, (kh*3+kw)*C + c]  (Eq. 3 for a
    convolution; out-of-range x is 0).  x_bits: bf16 bit patterns NB x H x W x C.  float64 result."""
    NB, H, Wd, C = x_bits.shape
    I = W.shape[0]
    Ho, Wo = conv_out_size(H, stride), conv_out_size(Wd, stride)
    xp = _pad_hw(bf16_to_f64(x_bits).reshape(NB, H, Wd, C))
    Wf = (bf16_round(W) * B).reshape(I, 3, 3, C)
    y = np.zeros((NB, Ho, Wo, I))
    for kh in range(3):
        for kw in range(3):
            y += xp[:, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride, :] @ Wf[:, kh, kw, :].T
    return y


def conv_dgrad(dy_bits, W, M_b, C, stride=1, in_hw=None):
    """dx[n, h, w, c] = sum over (kh, kw, i) and output pixels (ho, wo) with ho*s+kh-1 = h, wo*s+kw-1 = w of
    dy[n, ho, wo, i] * (M_b.W)[i, (kh*3+kw)*C + c]: the input gradient of conv_fwd with the backward mask in place of
    the forward one (Eq. 8 / Eq. 10).  in_hw = (H, W) of x (needed when stride > 1)."""
    NB, Ho, Wo, I = dy_bits.shape
    H, Wd = in_hw if in_hw is not None else (Ho, Wo)
    dy = bf16_to_f64(dy_bits).reshape(NB, Ho, Wo, I)
    Wb = (bf16_round(W) * M_b).reshape(I, 3, 3, C)
    dxp = np.zeros((NB, H + 2, Wd + 2, C))                      # padded input gradient; the border is dropped
    for kh in range(3):
        for kw in range(3):
            dxp[:, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride, :] += dy @ Wb[:, kh, kw, :]
    return dxp[:, 1:H + 1, 1:Wd + 1, :]


def conv_wgrad(dy_bits, x_bits, stride=1):
    """dW[i, (kh*3+kw)*C + c] = sum_{n, ho, wo} dy[n, ho, wo, i] * x[n, ho*s+kh-1, wo*s+kw-1, c]  (dense, STE)."""
    NB, H, Wd, C = x_bits.shape
    _, Ho, Wo, I = dy_bits.shape
    xp = _pad_hw(bf16_to_f64(x_bits).reshape(NB, H, Wd, C))
    dy = bf16_to_f64(dy_bits).reshape(NB * Ho * Wo, I)
    dW = np.zeros((I, 3, 3, C))
    for kh in range(3):
        for kw in range(3):
            patch = xp[:, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride, :]
            dW[:, kh, kw, :] = dy.T @ patch.reshape(NB * Ho * Wo, C)
    return dW.reshape(I, 9 * C)


def conv_layer_step(W, x_bits, dy_bits, N, M, P, seed, do_search=True, perm=None, stride=1):
    """One iteration of Alg. 1 for a 3x3 convolution layer (padding 1, stride 1 or 2): masks and search exactly as
    for a linear layer on the I x 9C matrix view; the three products are convolutions."""
    NB, H, Wd, C = x_bits.shape
    assert W.shape[1] == 9 * C
    out = layer_step(W, None, None, N, M, P, seed, do_search=do_search, perm=perm, with_gemms=False)
    out["y"] = conv_fwd(x_bits, W, out["B"], stride)
    out["dx"] = conv_dgrad(dy_bits, W, out["M_b"], C, stride, (H, Wd))
    out["dW"] = conv_wgrad(dy_bits, x_bits, stride)
    return out


# ---------------------------------------------------------------------------------------
# Greedy refinement of a permutation (beyond the paper: its conclusion names a better search than
# "best of K random candidates" as future work).  Not part of Algorithm 1.
# ---------------------------------------------------------------------------------------
REFINE_SEED_OFFSET = 0x5EED5EED


def _block_eligible(B, rows, N):
    """Columns of the row block `rows` (M row indices of B) that hold at most N ones."""
    return int((B[np.asarray(rows, dtype=np.int64), :].sum(axis=0) <= N).sum())


def refine_perm(B, perm, N, M, rounds, seed):
    """Pairwise-swap hill climbing on the eligible-block count.  Round r pairs up the POSITIONS of the
    permutation at random: with order = candidates(seed + REFINE_SEED_OFFSET, rounds, I)[r], pair i is
    (a, b) = (order[2i], order[2i+1]).  A pair whose positions lie in different row blocks ka != kb
    has gain = (eligible columns of the two blocks after exchanging perm[a] and perm[b]) - (before),
    all gains taken against the permutation at the start of the round.  A pair is accepted when its
    gain is positive and, for BOTH of its blocks, it is the best pair touching that block (largest
    gain, lowest pair index on equal gain) -- so accepted pairs never share a block, their gains add
    up, and the count never decreases.  Returns (perm, eligible-block count of the result)."""
    perm = np.array(perm, dtype=np.int32).copy()
    I = perm.shape[0]
    assert I % M == 0
    orders = candidates((int(seed) + REFINE_SEED_OFFSET) & MASK64, rounds, I) if rounds > 0 else None
    for r in range(rounds):
        order = orders[r]
        gains = {}
        best = {}                                            # block -> (gain, -pair index) of its best pair
        for i in range(I // 2):
            a, b = int(order[2 * i]), int(order[2 * i + 1])
            ka, kb = a // M, b // M
            if ka == kb:
                continue
            rows_a = perm[ka * M:(ka + 1) * M].copy()
            rows_b = perm[kb * M:(kb + 1) * M].copy()
            before = _block_eligible(B, rows_a, N) + _block_eligible(B, rows_b, N)
            rows_a[a - ka * M], rows_b[b - kb * M] = perm[b], perm[a]
            gain = _block_eligible(B, rows_a, N) + _block_eligible(B, rows_b, N) - before
            if gain > 0:
                gains[i] = (gain, a, b, ka, kb)
                for k in (ka, kb):
                    if k not in best or (gain, -i) > best[k]:
                        best[k] = (gain, -i)
        for i, (gain, a, b, ka, kb) in gains.items():
            if best[ka] == (gain, -i) and best[kb] == (gain, -i):
                perm[a], perm[b] = perm[b], perm[a]
    return perm, eligible_blocks(B, perm, N, M)
