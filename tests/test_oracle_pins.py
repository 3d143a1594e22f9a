"""Pins for the CPU oracle: everything here checks oracle/ against something other than
itself -- hand-worked examples (tests/golden), brute force written a different way,
closed forms, invariants the paper states, and special cases that reduce to library
routines.  No GPU needed."""
import itertools
import math
import os

import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st

from oracle import bimask_oracle as O
from paper_2302_06058_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- golden readers
def _read_blocks():
    rows = []
    with open(os.path.join(GOLDEN, "handworked_blocks.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            n, w, kept, code, slots = [p.strip() for p in line.split("|")]
            rows.append((int(n), [float(x) for x in w.split()], [int(x) for x in kept.split()],
                         int(code, 16), [float(x) for x in slots.split()]))
    return rows


def _read_example():
    sections = {}
    cur = None
    with open(os.path.join(GOLDEN, "example_8x8.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("["):
                cur = line
                sections[cur] = []
            else:
                sections[cur].append(line)
    W = np.array([[float(x) for x in r.split()] for r in sections["[W]"]], dtype=np.float32)
    B = np.array([[int(x) for x in r.split()] for r in sections["[B]"]], dtype=bool)
    perms = []
    for r in sections["[perm count nnz(B-bar)]"]:
        p, c, n = [q.strip() for q in r.split("|")]
        perms.append(([int(x) for x in p.split()], int(c), int(n)))
    global EXAMPLE_HISTOGRAM
    EXAMPLE_HISTOGRAM = {int(r.split()[0]): int(r.split()[1]) for r in sections["[histogram count orders]"]}
    return W, B, perms


# ---------------------------------------------------------------- independent brute force
def brute_forward_mask(W, N, M):
    """Top-N per block by sorting (-|w|, index): a different formulation of Eq. 4."""
    I, J = W.shape
    B = np.zeros((I, J), dtype=bool)
    for i in range(I):
        for g in range(J // M):
            blk = [(-abs(float(W[i, g * M + m])), m) for m in range(M)]
            for _, m in sorted(blk)[:N]:
                B[i, g * M + m] = True
    return B


def brute_backward_mask(W, B, perm, N, M):
    """Eq. 11 by sorting, on (B*W)[perm, :] restricted to forward survivors."""
    I, J = W.shape
    out = np.zeros((I, J), dtype=bool)
    for l in range(J):
        for k in range(I // M):
            blk = [(-abs(float(W[perm[k * M + m], l])), m) for m in range(M) if B[perm[k * M + m], l]]
            for _, m in sorted(blk)[:N]:
                out[k * M + m, l] = True
    return out


def brute_count(B, perm, N, M):
    I, J = B.shape
    total = 0
    for k in range(I // M):
        for l in range(J):
            s = 0
            for m in range(M):
                s += 1 if B[perm[k * M + m], l] else 0
            total += 1 if s <= N else 0
    return total


# ---------------------------------------------------------------- hand-worked examples
@pytest.mark.parametrize("row", _read_blocks())
def test_handworked_block(row):
    n, w, kept, code, slots = row
    # a full 32-wide row so that the packed format applies; the block under test is group 0,
    # the other groups are copies (every group packs independently)
    W = np.tile(np.array(w, dtype=np.float32), 8)[None, :]
    B = O.forward_mask(W, n, 4)
    assert list(np.nonzero(B[0, :4])[0]) == kept
    vals, meta = O.pack_2to4(W, B)
    assert (int(meta[0, 0]) & 0xF) == code
    assert int(meta[0, 0]) == sum(code << (4 * g) for g in range(8))
    got = O.bf16_to_f64(vals[0, :2])
    assert all((np.isnan(g) and np.isnan(s)) or (g == s and np.signbit(g) == np.signbit(s)) or
               (s == 0 and g == 0 and not any(np.signbit(x) for x in w)) for g, s in zip(got, slots)), (got, slots)
    if any(np.isnan(x) for x in w):                        # the quiet-NaN pattern of the conversion rule
        nan_slot = [i for i, s in enumerate(slots) if np.isnan(s)][0]
        assert int(vals[0, nan_slot]) == 0x7FC0


def test_two_blocks_share_a_byte():
    W = np.tile(np.array([9, -1, 4, -6, 2, 7, -3, 5], dtype=np.float32), 4)[None, :]
    B = O.forward_mask(W, 2, 4)
    _, meta = O.pack_2to4(W, B)
    assert (int(meta[0, 0]) & 0xFF) == 0xDC          # block 0 in the low nibble
    bits = O.pack_bits(B)
    assert (int(bits[0, 0]) & 0xFF) == 0b10101001    # bit j of the word = column j


def test_example_8x8_mask_and_counts():
    W, B, perms = _read_example()
    assert np.array_equal(O.forward_mask(W, 2, 4), B)
    for p, count, nnz in perms:
        assert O.eligible_blocks(B, np.array(p), 2, 4) == count
        Bbar = O.backward_mask(W, B, np.array(p), 2, 4)
        assert int(Bbar.sum()) == nnz
        assert np.array_equal(Bbar, brute_backward_mask(W, B, p, 2, 4))


def test_example_8x8_all_permutations():
    """All 8! row orders: the oracle's count equals a plain triple loop, and the search over
    all of them returns the first maximiser."""
    W, B, _ = _read_example()
    allp = np.array(list(itertools.permutations(range(8))), dtype=np.int32)
    ref = np.array([brute_count(B, p, 2, 4) for p in allp])
    best, best_perm, counts = O.perm_search(B, allp, 2, 4)
    assert np.array_equal(counts, ref)
    assert counts.max() == 16 and counts.min() == 8
    assert best == int(np.nonzero(ref == 16)[0][0])
    assert np.array_equal(best_perm, allp[best])
    # the count depends only on which rows share a block: 8!/(4!4!2) = 35 splits, each hit 1152 times
    hist = {int(v): int((ref == v).sum()) for v in np.unique(ref)}
    assert all(n % 1152 == 0 for n in hist.values())
    assert sum(hist.values()) == math.factorial(8)
    assert hist == EXAMPLE_HISTOGRAM                      # the hand-tallied histogram of the fixture


# ---------------------------------------------------------------- brute force on random inputs
@pytest.mark.parametrize("N,M", [(2, 4), (1, 4), (3, 4), (4, 4), (2, 8), (4, 8), (1, 16)])
def test_masks_match_sort_based_definition(N, M):
    rng = np.random.default_rng(5)
    I, J = 2 * M * 2, 32 * max(1, M // 4)
    # few distinct magnitudes => many ties, plus exact zeros and negative zero
    W = rng.integers(-3, 4, size=(I, J)).astype(np.float32)
    W[0, :4] = [-0.0, 0.0, 0.0, -0.0]
    B = O.forward_mask(W, N, M)
    assert np.array_equal(B, brute_forward_mask(W, N, M))
    perm = rng.permutation(I)
    Bbar = O.backward_mask(W, B, perm, N, M)
    assert np.array_equal(Bbar, brute_backward_mask(W, B, perm, N, M))
    assert O.eligible_blocks(B, perm, N, M) == brute_count(B, perm, N, M)


def test_literal_eq4_agrees_when_magnitudes_distinct():
    """Eq. 4 verbatim (zero iff |w| < N-th largest of the block) on tie-free weights."""
    rng = np.random.default_rng(11)
    W = rng.standard_normal((16, 64)).astype(np.float32)
    for N, M in [(2, 4), (1, 4), (2, 8)]:
        blocks = np.abs(W).reshape(16, 64 // M, M)
        nth = np.sort(blocks, axis=2)[:, :, M - N][:, :, None]
        literal = (blocks >= nth).reshape(16, 64)
        assert np.array_equal(O.forward_mask(W, N, M), literal)


def test_literal_eq9_agrees_when_magnitudes_distinct():
    rng = np.random.default_rng(12)
    W = rng.standard_normal((16, 32)).astype(np.float32)
    B = O.forward_mask(W, 2, 4)
    masked = np.abs(W) * B
    blocks = masked.reshape(4, 4, 32)                       # (block, m, column)
    nth = np.sort(blocks, axis=1)[:, 2, :][:, None, :]      # 2nd largest of 4
    literal = np.where(blocks < nth, False, B.reshape(4, 4, 32)).reshape(16, 32)
    got = O.backward_mask(W, B, np.arange(16), 2, 4)
    assert np.array_equal(got, literal)


# ---------------------------------------------------------------- invariants
@settings(max_examples=40, deadline=None)
@given(st.integers(0, 2**31 - 1), st.sampled_from([(2, 4), (1, 4), (2, 8), (1, 8)]),
       st.integers(1, 3), st.integers(1, 2))
def test_invariants(seed, nm, ib, jb):
    N, M = nm
    I, J = 8 * ib * (M // 4), 32 * jb
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((I, J)).astype(np.float32)
    W[rng.random((I, J)) < 0.1] = 0.0
    B = O.forward_mask(W, N, M)
    assert (B.reshape(I, J // M, M).sum(axis=2) == N).all()                 # Eq. 2, exactly N
    perm = rng.permutation(I).astype(np.int32)
    Bbar = O.backward_mask(W, B, perm, N, M)
    Bp = B[perm]
    assert not (Bbar & ~Bp).any()                                            # B = 0 => B-bar = 0
    pop_f = Bp.reshape(I // M, M, J).sum(axis=1)
    pop_b = Bbar.reshape(I // M, M, J).sum(axis=1)
    assert (pop_b <= N).all()                                                # Eq. 7
    assert np.array_equal(pop_b, np.minimum(pop_f, N))
    same = (Bbar.reshape(I // M, M, J) == Bp.reshape(I // M, M, J)).all(axis=1)
    assert np.array_equal(same, pop_f <= N)          # eligible block <=> B-bar block == B block
    assert O.eligible_blocks(B, perm, N, M) == int(same.sum())
    Mb = O.unpermute_rows(Bbar, perm)
    assert np.array_equal(Mb[perm], Bbar)
    if M == 4:
        vals, meta = O.pack_2to4(W, B)
        vf, mf = O.pack_2to4_fast(W, B)
        assert np.array_equal(vals, vf) and np.array_equal(meta, mf)
        codes = (meta[:, :, None] >> (4 * np.arange(8, dtype=np.uint32))) & 0xF
        assert np.isin(codes, [0x4, 0x8, 0xC, 0x9, 0xD, 0xE]).all()
        assert np.array_equal(O.unpack_2to4(vals, meta), O.bf16_round(W) * B)
        assert np.array_equal(O.unpack_bits(O.pack_bits(B), J), B)
        if I % 32 == 0:
            _, vb, mb = O.backward_operand(W, Bbar, perm)
            vb2, mb2 = O.pack_2to4(np.ascontiguousarray(W[perm].T), np.ascontiguousarray(Bbar.T))
            assert np.array_equal(vb, vb2) and np.array_equal(mb, mb2)
            assert np.array_equal(O.unpack_2to4(vb, mb), (O.bf16_round(W)[perm] * Bbar).T)


# ---------------------------------------------------------------- closed forms
@pytest.mark.parametrize("N,M,elig,ratio", [(2, 4, 11 / 16, 13 / 16), (1, 4, 189 / 256, 175 / 256),
                                            (4, 8, 163 / 256, None), (2, 8, 0.6785431, None), (1, 16, 0.7358865, None)])
def test_closed_form_eligible_fraction(N, M, elig, ratio):
    """For i.i.d. continuous weights the forward bits of one column over distinct rows are
    i.i.d. Bernoulli(N/M): P(eligible) = P(Bin(M, N/M) <= N), E nnz(B-bar)/nnz(B) =
    E min(Bin, N) / N."""
    binom = [math.comb(M, k) * (N / M) ** k * (1 - N / M) ** (M - k) for k in range(M + 1)]
    assert abs(sum(binom[:N + 1]) - elig) < 1e-6
    if ratio is None:
        ratio = sum(min(k, N) * binom[k] for k in range(M + 1)) / N
    assert abs(sum(min(k, N) * binom[k] for k in range(M + 1)) / N - ratio) < 1e-12
    W = inputs.make_weight(512, 1024, 7)
    B = O.forward_mask(W, N, M)
    perm = np.random.default_rng(3).permutation(512)
    nblocks = (512 // M) * 1024
    frac = O.eligible_blocks(B, perm, N, M) / nblocks
    sigma = math.sqrt(elig * (1 - elig) / nblocks)
    assert abs(frac - elig) < 6 * sigma
    Bbar = O.backward_mask(W, B, perm, N, M)
    assert abs(Bbar.sum() / B.sum() - ratio) < 5e-3


# ---------------------------------------------------------------- special cases -> library routines
def test_n_equals_m_reduces_to_plain_matmul():
    W, X, dY = inputs.make_layer(1, 0, T=48)
    out = O.layer_step(W, X, dY, 4, 4, 2, 1)
    assert out["B"].all() and out["Bbar_p"].all()
    Wt = torch.from_numpy(W).to(torch.bfloat16).to(torch.float64)
    Xt = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).to(torch.float64)
    dYt = torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).to(torch.float64)
    assert np.allclose(out["Y"], (Xt @ Wt.T).numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(out["dX"], (dYt @ Wt).numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(out["dW"], (dYt.T @ Xt).numpy(), rtol=1e-12, atol=1e-12)


def test_masked_products_against_torch():
    W, X, dY = inputs.make_layer(1, 0, T=40)
    out = O.layer_step(W, X, dY, 2, 4, 8, 43)
    Wt = torch.from_numpy(W).to(torch.bfloat16).to(torch.float64)
    Xt = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).to(torch.float64)
    dYt = torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).to(torch.float64)
    Bf = torch.from_numpy(brute_forward_mask(W, 2, 4)).to(torch.float64)
    assert np.allclose(out["Y"], (Xt @ (Wt * Bf).T).numpy(), rtol=1e-12, atol=1e-12)
    Mb = torch.from_numpy(out["M_b"]).to(torch.float64)
    assert np.allclose(out["dX"], (dYt @ (Wt * Mb)).numpy(), rtol=1e-12, atol=1e-12)
    assert np.allclose(out["dW"], (dYt.T @ Xt).numpy(), rtol=1e-12, atol=1e-12)
    # transposition check: Y is T x I, dX is T x J, dW is I x J
    assert out["Y"].shape == (40, 256) and out["dX"].shape == (40, 256) and out["dW"].shape == (256, 256)


def test_permuted_form_equals_unpermuted_form():
    """Eq. 10: permuting W's rows and dY's columns together leaves the product unchanged."""
    W, X, dY = inputs.make_layer(1, 0, T=32)
    B = O.forward_mask(W, 2, 4)
    perm = O.candidates(9, 1, 256)[0]
    Bbar = O.backward_mask(W, B, perm, 2, 4)
    a = O.spmm_dgrad(dY, W, O.unpermute_rows(Bbar, perm))
    b = O.spmm_dgrad_permuted(dY, W, Bbar, perm)
    assert np.allclose(a, b, rtol=1e-12, atol=1e-12)


def test_planted_transposable_mask_gives_exact_gradient():
    """If every column block of B[perm] is already N:M, B-bar = B[perm], every block is
    eligible and Eq. 10 equals the exact gradient of Eq. 5."""
    for N in (2, 1):
        W, Q = inputs.planted_transposable(64, 96, N, 4, 21)
        B = O.forward_mask(W, N, 4)
        rng = np.random.default_rng(0)
        cands = np.stack([rng.permutation(64) for _ in range(5)] + [Q] +
                         [rng.permutation(64) for _ in range(3)]).astype(np.int32)
        best, perm, counts = O.perm_search(B, cands, N, 4)
        assert best == 5 and counts[5] == (64 // 4) * 96 and (counts[:5] < counts[5]).all()
        Bbar = O.backward_mask(W, B, perm, N, 4)
        assert np.array_equal(Bbar, B[perm])
        dY = inputs.make_activation(24, 64, 3)
        exact = O.dense_dgrad(dY, W, B)
        approx = O.spmm_dgrad(dY, W, O.unpermute_rows(Bbar, perm))
        assert np.allclose(exact, approx, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- bf16 rounding, generator
def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.standard_normal(100000).astype(np.float32),
                        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, np.inf, -np.inf,
                                  3.3895314e38, 1e-40, -1e-40, 65504.0], dtype=np.float32),
                        # exact ties: mantissa ends in 0x8000
                        (np.arange(0x3F800000, 0x3F800000 + 64 * 0x8000, 0x8000, dtype=np.uint32)).view(np.float32)])
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.bf16_bits(x), ref)
    assert np.array_equal(O.bf16_to_f64(ref), torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy())
    nan = O.bf16_bits(np.array([np.nan], dtype=np.float32))
    assert (int(nan[0]) & 0x7F80) == 0x7F80 and (int(nan[0]) & 0x7F) != 0


def test_mixer_matches_splitmix64_test_vector():
    """mix64(seed + golden gamma) is SplitMix64's output function; its published outputs for
    seed 0 are e220a8397b1dcdaf, 6e789e6aa1b965f4, 06c45d188009454f."""
    g = 0x9E3779B97F4A7C15
    got = [O._mix64((k * g) & O.MASK64) for k in (1, 2, 3)]
    assert got == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]
    z = np.array([(k * g) & O.MASK64 for k in (1, 2, 3)], dtype=np.uint64)
    with np.errstate(over="ignore"):
        assert [int(v) for v in O._mix64_np(z)] == got


def test_candidates_are_permutations_and_uniform():
    c = O.candidates(42, 16, 1000)
    assert c.shape == (16, 1000) and c.dtype == np.int32
    for row in c:
        assert np.array_equal(np.sort(row), np.arange(1000))
    assert len({tuple(r) for r in c}) == 16
    assert np.array_equal(O.candidates(42, 16, 1000)[3], c[3])          # deterministic
    assert not np.array_equal(O.candidates(43, 1, 1000)[0], c[0])       # seed matters
    # position x value chi-square on many small permutations (49 degrees of freedom)
    n = 20000
    small = O.candidates(7, n, 8)
    table = np.zeros((8, 8))
    for pos in range(8):
        table[pos] = np.bincount(small[:, pos], minlength=8)
    chi2 = ((table - n / 8) ** 2 / (n / 8)).sum()
    assert chi2 < 49 + 6 * math.sqrt(2 * 49)
    # independent restatement of the key construction for one candidate, in Python integers
    seed, cidx, I = 42, 2, 50
    stream = O._mix64((seed + 0x9E3779B97F4A7C15 * (cidx + 1)) & O.MASK64)
    keys = sorted(((O._mix64(stream ^ i) & ~0xFFFFFF) | i) for i in range(I))
    assert [k & 0xFFFFFF for k in keys] == list(O.candidates(seed, 3, I)[2])


def test_candidates_match_the_independent_test_vector():
    """Seed 42, I = 8: the first three candidates as computed, independently of this oracle, from the written
    definition of the generator when the interface was drawn up."""
    want = [[5, 4, 2, 3, 7, 0, 1, 6], [2, 5, 6, 7, 0, 1, 3, 4], [7, 0, 2, 1, 5, 4, 6, 3]]
    assert O.candidates(42, 3, 8).tolist() == want


def test_layer_step_identity_when_not_searching():
    W, X, dY = inputs.make_layer(1, 0, T=8)
    out = O.layer_step(W, X, dY, 2, 4, 8, 43, do_search=False)
    assert np.array_equal(out["perm"], np.arange(256))
    out2 = O.layer_step(W, X, dY, 2, 4, 8, 43, do_search=True)
    assert out2["counts"].shape == (8,)
    assert out2["counts"][out2["best_idx"]] == out2["counts"].max()
    assert np.array_equal(out2["perm"], O.candidates(43, 8, 256)[out2["best_idx"]])


# ---------------------------------------------------------------- optimizer update, Delta-T schedule
def test_sgd_update_matches_torch_optimizer():
    """Library pin: torch.optim.SGD (momentum, weight decay, no dampening, no Nesterov) on the same
    float32 data; it may fuse multiply-adds, hence a few-ulp tolerance rather than equality."""
    rng = np.random.default_rng(3)
    W0 = rng.standard_normal((16, 24)).astype(np.float32)
    lr, mu, wd = 0.1, 0.9, 5e-4
    p = torch.nn.Parameter(torch.from_numpy(W0.copy()))
    opt = torch.optim.SGD([p], lr=lr, momentum=mu, weight_decay=wd)
    W, mom = W0.copy(), np.zeros_like(W0)
    for step in range(5):
        g = rng.standard_normal(W0.shape).astype(np.float32)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        W, mom = O.sgd_update(W, g, mom, lr, mu, wd)
        assert W.dtype == np.float32 and mom.dtype == np.float32
        assert np.allclose(W, p.detach().numpy(), rtol=2e-6, atol=2e-7), step


def test_sgd_update_closed_forms():
    """Dyadic numbers make every float32 operation exact, so the closed forms hold bit for bit:
    plain SGD sums the gradients; a constant gradient with momentum mu moves the weight by
    lr * g * sum_{k=1..n} (1 - mu^k) / (1 - mu); weight decay alone scales by (1 - lr*wd)^n."""
    W0 = np.array([[1.0, -2.0, 0.5, 8.0]], dtype=np.float32)
    g = np.array([[0.25, -0.5, 1.0, 2.0]], dtype=np.float32)
    W, mom = W0.copy(), np.zeros_like(W0)
    for _ in range(6):
        W, mom = O.sgd_update(W, g, mom, 0.5, 0.0, 0.0)
    assert np.array_equal(W, W0 - 6 * 0.5 * g)
    W, mom = W0.copy(), np.zeros_like(W0)
    n, mu, lr = 5, 0.5, 0.25
    for _ in range(n):
        W, mom = O.sgd_update(W, g, mom, lr, mu, 0.0)
    coef = sum((1 - mu ** k) / (1 - mu) for k in range(1, n + 1))
    assert np.array_equal(W, (W0 - lr * coef * g).astype(np.float32))
    assert np.array_equal(mom, g * np.float32((1 - mu ** n) / (1 - mu)))
    W, mom = W0.copy(), np.zeros_like(W0)
    for _ in range(3):
        W, mom = O.sgd_update(W, np.zeros_like(W0), mom, 0.5, 0.0, 0.25)
    assert np.array_equal(W, W0 * np.float32((1 - 0.125) ** 3))
    # the sign of each term: a positive gradient lowers the weight, decay pulls towards zero
    W1, _ = O.sgd_update(W0, g, np.zeros_like(W0), 0.5, 0.0, 0.0)
    assert np.all(np.sign(W1 - W0) == -np.sign(g))


def test_train_steps_schedule_and_return_value():
    """Algorithm 1's loop: the search runs exactly when t % Delta T == 0, with a fresh draw per
    interval; before it the permutation is the identity; every iteration sees the weights the
    previous update left; the return value is N:M sparse along each row."""
    N, M, P, seed, dT, iters = 2, 4, 6, 11, 3, 7
    rng = np.random.default_rng(5)
    W0 = rng.standard_normal((32, 32)).astype(np.float32)
    X = O.bf16_bits(rng.integers(-3, 4, size=(8, 32)).astype(np.float32))
    dY = [O.bf16_bits(rng.integers(-3, 4, size=(8, 32)).astype(np.float32)) for _ in range(iters)]
    hist, Wf, momf, sparse = O.train_steps(W0, X, dY, N, M, P, seed, dT, iters, 0.125, 0.5, 0.0)
    assert [h["searched"] for h in hist] == [False, False, True, False, False, True, False]
    ident = np.arange(32)
    assert np.array_equal(hist[0]["perm"], ident) and np.array_equal(hist[1]["perm"], ident)
    best, perm3, _ = O.perm_search(hist[2]["B"], O.candidates(seed + 1, P, 32), N, M)
    assert np.array_equal(hist[2]["perm"], perm3) and hist[2]["best_idx"] == best
    assert np.array_equal(hist[3]["perm"], perm3) and np.array_equal(hist[4]["perm"], perm3)
    best6, perm6, _ = O.perm_search(hist[5]["B"], O.candidates(seed + 2, P, 32), N, M)
    assert np.array_equal(hist[5]["perm"], perm6) and np.array_equal(hist[6]["perm"], perm6)
    # the chain of weights, replayed by hand from the recorded gradients (integers: exact)
    W, mom = W0.copy(), np.zeros_like(W0)
    for t, h in enumerate(hist):
        assert np.array_equal(h["W"], W), t
        assert np.array_equal(h["B"], O.forward_mask(W, N, M))
        dW = (O.bf16_to_f64(dY[t]).T @ O.bf16_to_f64(X)).astype(np.float32)
        assert np.array_equal(dW, h["dW"])
        mom = np.float32(0.5) * mom + dW
        W = W - np.float32(0.125) * mom
    assert np.array_equal(W, Wf) and np.array_equal(mom, momf)
    assert np.all((sparse != 0).reshape(32, 8, 4).sum(axis=2) <= N)
    assert np.array_equal(sparse != 0, O.forward_mask(Wf, N, M) & (Wf != 0))
    # lr = 0 freezes the weights: every iteration reproduces the first one's masks
    hist0, W_same, _, _ = O.train_steps(W0, X, dY[0], N, M, P, seed, dT, 4, 0.0, 0.9, 0.0)
    assert np.array_equal(W_same, W0)
    assert all(np.array_equal(h["B"], hist0[0]["B"]) for h in hist0)


# ---------------------------------------------------------------- backward-mask criteria (ablation variants)
def _all_valid_case(a_rows, nblocks, J):
    """W whose every block of 4 permuted rows holds the magnitudes a_rows in every column; B all ones."""
    W = np.tile(np.asarray(a_rows, dtype=np.float32)[:, None], (nblocks, J))
    W *= np.where(np.arange(W.shape[0])[:, None] % 3 == 0, -1.0, 1.0).astype(np.float32)   # signs must not matter
    return W, np.ones(W.shape, dtype=bool), np.arange(W.shape[0])


def _subset_histogram(Bbar, nblocks, J):
    code = (Bbar.reshape(nblocks, 4, J) * np.array([1, 2, 4, 8])[None, :, None]).sum(axis=1)
    assert set(np.unique(code)) <= {3, 5, 6, 9, 10, 12}                                      # exactly two kept
    return {c: int((code == c).sum()) for c in (3, 5, 6, 9, 10, 12)}


def test_criterion_score_is_the_rank_rule_on_another_matrix():
    rng = np.random.default_rng(21)
    for (N, M) in [(2, 4), (1, 4), (2, 8), (4, 8)]:
        W = rng.standard_normal((32, 16)).astype(np.float32)
        S = rng.standard_normal((32, 16)).astype(np.float32)
        S[3, :] = S[7, :]                                            # ties between rows of one block
        B = O.forward_mask(W, N, M)
        perm = rng.permutation(32)
        assert np.array_equal(O.backward_mask_criterion(W, B, perm, N, M, O.CRIT_SCORE, S=W),
                              O.backward_mask(W, B, perm, N, M))
        got = O.backward_mask_criterion(W, B, perm, N, M, O.CRIT_SCORE, S=S)
        Sp, Bp = np.abs(S[perm]), B[perm]
        for k0 in range(0, 32, M):
            for l in range(16):
                comp = [m for m in range(M) if Bp[k0 + m, l]]
                order = sorted(comp, key=lambda m: (-Sp[k0 + m, l], m))[:N]
                want = np.zeros(M, dtype=bool)
                want[order] = True
                assert np.array_equal(got[k0:k0 + M, l], want)


def test_criterion_random_is_uniform_over_subsets():
    nblocks, J = 512, 64
    W, B, perm = _all_valid_case([1.0, 2.0, 3.0, 4.0], nblocks, J)
    got = O.backward_mask_criterion(W, B, perm, 2, 4, O.CRIT_RANDOM, seed=99)
    hist = _subset_histogram(got, nblocks, J)
    n = nblocks * J
    chi2 = sum((v - n / 6) ** 2 / (n / 6) for v in hist.values())
    assert chi2 < 5 + 6 * math.sqrt(2 * 5)
    assert not np.array_equal(got, O.backward_mask_criterion(W, B, perm, 2, 4, O.CRIT_RANDOM, seed=100))
    # the key belongs to the weight, not to its position: permuting rows permutes the keys with them
    k = O.random_keys(99, 8, 4)
    assert k.min() >= 0 and k.max() < 2 ** 31 and len(np.unique(k)) == 32


def test_criterion_multinomial_matches_exact_subset_probabilities():
    """Two draws without replacement, each proportional to |w|: P{i,j} = p_i p_j/(1-p_i) + p_j p_i/(1-p_j)."""
    nblocks, J = 1024, 64
    a = [1.0, 2.0, 3.0, 4.0]
    W, B, perm = _all_valid_case(a, nblocks, J)
    got = O.backward_mask_criterion(W, B, perm, 2, 4, O.CRIT_MULTINOMIAL, seed=5)
    hist = _subset_histogram(got, nblocks, J)
    p = np.array(a) / sum(a)
    n = nblocks * J
    chi2 = 0.0
    for i, j in itertools.combinations(range(4), 2):
        prob = p[i] * p[j] / (1 - p[i]) + p[j] * p[i] / (1 - p[j])
        chi2 += (hist[(1 << i) | (1 << j)] - n * prob) ** 2 / (n * prob)
    assert chi2 < 5 + 6 * math.sqrt(2 * 5)


def test_criterion_multinomial_first_draw_is_the_inverse_cdf_and_special_cases():
    nblocks, J = 64, 32
    W, B, perm = _all_valid_case([1.0, 1.0, 2.0, 4.0], nblocks, J)      # running sums 1, 2, 4, 8: exact
    got = O.backward_mask_criterion(W, B, perm, 1, 4, O.CRIT_MULTINOMIAL, seed=8)
    idx = np.arange(nblocks, dtype=np.uint64)[:, None] * np.uint64(J) + np.arange(J, dtype=np.uint64)[None, :]
    u = O._uniform24(8, 0, idx).astype(np.float64)
    assert u.min() >= 0 and u.max() < 1 and abs(u.mean() - 0.5) < 0.03
    want = np.searchsorted(np.array([1.0, 2.0, 4.0, 8.0]), 8 * u.ravel(), side="right").reshape(nblocks, J)
    assert np.array_equal(np.argmax(got.reshape(nblocks, 4, J), axis=1), want)
    assert np.all(got.reshape(nblocks, 4, J).sum(axis=1) == 1)
    # a weight that dwarfs the rest is always drawn; zero weights are drawn only when nothing else is left
    W2, B2, perm2 = _all_valid_case([1e-30, 0.0, 1e30, 0.0], 16, 32)
    g2 = O.backward_mask_criterion(W2, B2, perm2, 2, 4, O.CRIT_MULTINOMIAL, seed=1).reshape(16, 4, 32)
    assert g2[:, 2].all() and g2[:, 0].all() and not g2[:, 1].any() and not g2[:, 3].any()
    W3, B3, perm3 = _all_valid_case([0.0, 0.0, 0.0, 0.0], 4, 32)
    g3 = O.backward_mask_criterion(W3, B3, perm3, 2, 4, O.CRIT_MULTINOMIAL, seed=1).reshape(4, 4, 32)
    assert g3[:, 0].all() and g3[:, 1].all() and not g3[:, 2:].any()


@pytest.mark.parametrize("crit", [1, 2, 3])
def test_criteria_keep_the_structure_of_eq11(crit):
    """Whatever the criterion: a subset of B[perm], min(N, competitors) survivors per block, and
    blocks with at most N competitors are untouched (no gradient gap there)."""
    rng = np.random.default_rng(crit)
    for (N, M) in [(2, 4), (1, 4), (2, 8), (1, 16), (4, 8)]:
        W = rng.standard_normal((64, 32)).astype(np.float32)
        B = O.forward_mask(W, N, M)
        perm = rng.permutation(64)
        got = O.backward_mask_criterion(W, B, perm, N, M, crit, S=rng.standard_normal((64, 32)).astype(np.float32), seed=3)
        Bp = B[perm]
        assert not (got & ~Bp).any()
        comp = Bp.reshape(64 // M, M, 32).sum(axis=1)
        assert np.array_equal(got.reshape(64 // M, M, 32).sum(axis=1), np.minimum(comp, N))


def test_dense_operand_agrees_with_the_packed_one():
    """For a packable pattern the dense masked operand is what the 2:4 operand expands to; for 4:8 it
    carries exactly the kept weights (bf16) and zeros, and the products computed from it are Eq. 3 / Eq. 10."""
    rng = np.random.default_rng(31)
    W = rng.standard_normal((32, 64)).astype(np.float32)
    B = O.forward_mask(W, 2, 8)
    vals, meta = O.pack_2to4(W, B)
    assert np.array_equal(O.bf16_to_f64(O.dense_operand(W, B)), O.unpack_2to4(vals, meta))
    B48 = O.forward_mask(W, 4, 8)
    D = O.dense_operand(W, B48)
    assert np.array_equal(D != 0, B48 & (O.bf16_bits(W) != 0))
    assert np.array_equal(D[B48], O.bf16_bits(W)[B48])
    X = O.bf16_bits(rng.standard_normal((8, 64)).astype(np.float32))
    assert np.allclose(O.bf16_to_f64(X) @ O.bf16_to_f64(D).T, O.spmm_fwd(X, W, B48), rtol=1e-12, atol=1e-12)
    perm = rng.permutation(32)
    Bbar = O.backward_mask(W, B48, perm, 4, 8)
    Db = O.dense_backward_operand(W, Bbar, perm)
    assert Db.shape == (64, 32)
    dY = O.bf16_bits(rng.standard_normal((8, 32)).astype(np.float32))
    want = O.spmm_dgrad(dY, W, O.unpermute_rows(Bbar, perm))
    assert np.allclose(O.bf16_to_f64(dY)[:, perm] @ O.bf16_to_f64(Db).T, want, rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- convolution layer
def test_conv_products_match_torch_conv2d_and_autograd():
    """Library pin: torch's conv2d (float64) and its autograd for the two gradients, on bf16-valued data."""
    rng = np.random.default_rng(41)
    NB, H, Wd, C, I = 2, 5, 6, 8, 12
    W = rng.standard_normal((I, 9 * C)).astype(np.float32)
    B = O.forward_mask(W, 2, 4)
    perm = rng.permutation(I)
    M_b = O.unpermute_rows(O.backward_mask(W, B, perm, 2, 4), perm)
    x = O.bf16_bits(rng.standard_normal((NB, H, Wd, C)).astype(np.float32))
    dy = O.bf16_bits(rng.standard_normal((NB, H, Wd, I)).astype(np.float32))

    def filt(mask):        # I x (kh, kw, c)  ->  torch's I x C x kh x kw
        return torch.from_numpy((O.bf16_round(W) * mask).reshape(I, 3, 3, C)).permute(0, 3, 1, 2).contiguous()

    xt = torch.from_numpy(O.bf16_to_f64(x).reshape(NB, H, Wd, C)).permute(0, 3, 1, 2).contiguous().requires_grad_(True)
    dyt = torch.from_numpy(O.bf16_to_f64(dy).reshape(NB, H, Wd, I)).permute(0, 3, 1, 2).contiguous()
    y = torch.nn.functional.conv2d(xt, filt(B), padding=1)
    assert np.allclose(O.conv_fwd(x, W, B), y.detach().permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    # input gradient through the BACKWARD mask: differentiate a convolution whose filter is M_b . W
    wb = filt(M_b)
    (gx,) = torch.autograd.grad(torch.nn.functional.conv2d(xt, wb, padding=1), xt, dyt)
    assert np.allclose(O.conv_dgrad(dy, W, M_b, C), gx.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    # dense weight gradient
    wd = filt(np.ones_like(B)).requires_grad_(True)
    (gw,) = torch.autograd.grad(torch.nn.functional.conv2d(xt.detach(), wd, padding=1), wd, dyt)
    assert np.allclose(O.conv_wgrad(dy, x), gw.permute(0, 2, 3, 1).reshape(I, 9 * C).numpy(), rtol=1e-12, atol=1e-12)


def test_conv_equals_the_linear_layer_on_the_column_matrix():
    """im2col identity: the convolution is the linear layer applied to the T x 9C matrix of shifted pixels."""
    rng = np.random.default_rng(43)
    NB, H, Wd, C, I = 2, 4, 4, 32, 32
    W = rng.standard_normal((I, 9 * C)).astype(np.float32)
    x = O.bf16_bits(rng.standard_normal((NB, H, Wd, C)).astype(np.float32))
    dy = O.bf16_bits(rng.standard_normal((NB, H, Wd, I)).astype(np.float32))
    xp = np.pad(x, ((0, 0), (1, 1), (1, 1), (0, 0)))
    cols = np.concatenate([xp[:, kh:kh + H, kw:kw + Wd, :] for kh in range(3) for kw in range(3)], axis=3)
    Xcol = cols.reshape(NB * H * Wd, 9 * C)
    ref = O.layer_step(W, Xcol, dy.reshape(-1, I), 2, 4, 4, 3, do_search=True)
    got = O.conv_layer_step(W, x, dy, 2, 4, 4, 3, do_search=True)
    assert np.array_equal(got["perm"], ref["perm"]) and np.array_equal(got["B"], ref["B"])
    assert np.allclose(got["y"].reshape(-1, I), ref["Y"], rtol=1e-12, atol=1e-12)
    assert np.allclose(got["dW"], ref["dW"], rtol=1e-12, atol=1e-12)
    # dX of the linear layer lives in column space; folding it back (sum of the nine shifts) is dx
    dXcol = ref["dX"].reshape(NB, H, Wd, 9, C)
    dx = np.zeros((NB, H + 2, Wd + 2, C))
    for kh in range(3):
        for kw in range(3):
            dx[:, kh:kh + H, kw:kw + Wd, :] += dXcol[:, :, :, kh * 3 + kw, :]
    assert np.allclose(got["dx"], dx[:, 1:-1, 1:-1, :], rtol=1e-12, atol=1e-12)


# ---------------------------------------------------------------- greedy refinement of the permutation
def test_refine_perm_never_loses_and_matches_a_recount():
    """Every round's accepted swaps are re-derived here by brute force (full recount of the eligible blocks for
    each proposed swap), and the total must equal the sum of the accepted gains."""
    rng = np.random.default_rng(51)
    for (N, M, I, J) in [(2, 4, 32, 64), (1, 4, 32, 32), (2, 8, 64, 32)]:
        W = rng.standard_normal((I, J)).astype(np.float32)
        B = O.forward_mask(W, N, M)
        perm0 = rng.permutation(I).astype(np.int32)
        seed = 9
        counts = [O.eligible_blocks(B, perm0, N, M)]
        perm = perm0.copy()
        for r in range(1, 5):
            got, cnt = O.refine_perm(B, perm0, N, M, r, seed)
            assert np.array_equal(np.sort(got), np.arange(I)) and cnt == O.eligible_blocks(B, got, N, M)
            # one more round, by hand, from the previous result
            order = O.candidates(seed + O.REFINE_SEED_OFFSET, r, I)[r - 1]
            base = O.eligible_blocks(B, perm, N, M)
            cand = []
            for i in range(I // 2):
                a, b = int(order[2 * i]), int(order[2 * i + 1])
                if a // M == b // M:
                    continue
                q = perm.copy()
                q[a], q[b] = q[b], q[a]
                g = O.eligible_blocks(B, q, N, M) - base
                if g > 0:
                    cand.append((g, -i, a, b))
            accepted, nxt = [], perm.copy()
            for (g, ni, a, b) in cand:
                rivals = [c for c in cand if {c[2] // M, c[3] // M} & {a // M, b // M}]
                if all((g, ni) >= (c[0], c[1]) for c in rivals):
                    accepted.append(g)
                    nxt[a], nxt[b] = nxt[b], nxt[a]
            assert np.array_equal(nxt, got), (N, M, r)
            assert cnt == base + sum(accepted)
            counts.append(cnt)
            perm = nxt
        assert all(y >= x for x, y in zip(counts, counts[1:])) and counts[-1] > counts[0]


def test_refine_perm_fixed_point_and_improvement():
    # a permutation that already makes every block eligible cannot be improved
    W, Q = inputs.planted_transposable(64, 32, 2, 4, 3)
    B = O.forward_mask(W, 2, 4)
    assert O.eligible_blocks(B, Q, 2, 4) == (64 // 4) * 32
    got, cnt = O.refine_perm(B, Q, 2, 4, 6, 1)
    assert np.array_equal(got, Q) and cnt == 16 * 32
    # zero rounds: unchanged
    p = np.random.default_rng(1).permutation(64).astype(np.int32)
    got, cnt = O.refine_perm(B, p, 2, 4, 0, 1)
    assert np.array_equal(got, p)
    # i.i.d. weights: best-of-K sits at 11/16 of the blocks; hill climbing clearly beats it
    rng = np.random.default_rng(2)
    W = rng.standard_normal((128, 128)).astype(np.float32)
    B = O.forward_mask(W, 2, 4)
    best, perm, counts = O.perm_search(B, O.candidates(7, 16, 128), 2, 4)
    got, cnt = O.refine_perm(B, perm, 2, 4, 24, 7)
    total = (128 // 4) * 128
    assert abs(counts.mean() / total - 11 / 16) < 0.02
    assert cnt / total > 0.73 and cnt > counts.max() + 0.02 * total


def test_strided_conv_products_match_torch():
    """Stride 2 (ResNet's down-sampling 3x3 convolutions), odd and even image sizes, against torch and its autograd."""
    rng = np.random.default_rng(47)
    for (H, Wd) in [(6, 6), (7, 5)]:
        NB, C, I = 2, 8, 12
        W = rng.standard_normal((I, 9 * C)).astype(np.float32)
        B = O.forward_mask(W, 2, 4)
        perm = rng.permutation(I)
        M_b = O.unpermute_rows(O.backward_mask(W, B, perm, 2, 4), perm)
        Ho, Wo = O.conv_out_size(H, 2), O.conv_out_size(Wd, 2)
        x = O.bf16_bits(rng.standard_normal((NB, H, Wd, C)).astype(np.float32))
        dy = O.bf16_bits(rng.standard_normal((NB, Ho, Wo, I)).astype(np.float32))

        def filt(mask):
            return torch.from_numpy((O.bf16_round(W) * mask).reshape(I, 3, 3, C)).permute(0, 3, 1, 2).contiguous()

        xt = torch.from_numpy(O.bf16_to_f64(x).reshape(NB, H, Wd, C)).permute(0, 3, 1, 2).contiguous().requires_grad_(True)
        dyt = torch.from_numpy(O.bf16_to_f64(dy).reshape(NB, Ho, Wo, I)).permute(0, 3, 1, 2).contiguous()
        y = torch.nn.functional.conv2d(xt, filt(B), padding=1, stride=2)
        assert tuple(y.shape[2:]) == (Ho, Wo)
        assert np.allclose(O.conv_fwd(x, W, B, 2), y.detach().permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
        (gx,) = torch.autograd.grad(torch.nn.functional.conv2d(xt, filt(M_b), padding=1, stride=2), xt, dyt)
        assert np.allclose(O.conv_dgrad(dy, W, M_b, C, 2, (H, Wd)), gx.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
        wd = filt(np.ones_like(B)).requires_grad_(True)
        (gw,) = torch.autograd.grad(torch.nn.functional.conv2d(xt.detach(), wd, padding=1, stride=2), wd, dyt)
        assert np.allclose(O.conv_wgrad(dy, x, 2), gw.permute(0, 2, 3, 1).reshape(I, 9 * C).numpy(), rtol=1e-12, atol=1e-12)
