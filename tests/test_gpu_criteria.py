"""GPU parity for the backward mask under the ablation's other criteria (bimask_bwd_mask_criterion):
score matrix (gradient magnitude), multinomial draws, random.  Integer results: bit-exact."""
import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from tests.gpu_util import dev, u16, u32

pytestmark = pytest.mark.gpu

SHAPES = [(256, 256, 2, 4), (128, 384, 1, 4), (96, 160, 2, 4), (128, 128, 2, 8), (64, 96, 1, 8), (128, 64, 1, 16),
          (64, 64, 4, 8)]


def _case(I, J, N, M, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((I, J)) * 0.05).astype(np.float32)
    S = rng.standard_normal((I, J)).astype(np.float32)
    W[0:8, 0:4] = 0.25                  # equal magnitudes: ties under every criterion's rule
    W[8:16, 0:4] = 0.0                  # all-zero competitors: the multinomial fallback
    W[16:20, 1] = [np.inf, 1.0, -np.inf, 2.0]
    S[0:16, 0:4] = -1.5
    S[20:24, 2] = [0.0, -0.0, 0.0, -0.0]
    B = O.forward_mask(W, N, M)
    perm = rng.permutation(I).astype(np.int32)
    perm[:24] = np.arange(24)           # keep the planted rows together in their blocks
    rest = np.setdiff1d(np.arange(I), np.arange(24))
    perm[24:] = rng.permutation(rest)
    return W, S, B, perm


@pytest.mark.parametrize("I,J,N,M", SHAPES)
@pytest.mark.parametrize("crit", [0, 1, 2, 3])
def test_bwd_mask_criterion_bit_exact(I, J, N, M, crit):
    W, S, B, perm = _case(I, J, N, M, 100 + I + J + crit)
    seed = 1234 + crit
    pack = N <= 2
    b = bm.alloc_layer_buffers(1, I, J, 1)
    Wd, Sd, pd = dev(W), dev(S), dev(perm)
    bitsf = dev(O.pack_bits(B).view(np.int32))
    bm.bimask_bwd_mask_criterion(Wd, Sd if crit == 1 else None, bitsf, pd, I, J, N, M, crit, seed, b["maskbits_b"],
                                 b["vals_b"] if pack else None, b["meta_b"] if pack else None,
                                 b["hw_meta_b"] if pack else None)
    torch.cuda.synchronize()
    ref = O.backward_mask_criterion(W, B, perm, N, M, crit, S=S, seed=seed)
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(ref))
    if pack:
        _, vals, meta = O.backward_operand(W, ref, perm)
        assert np.array_equal(u16(b["vals_b"]), vals)
        assert np.array_equal(u32(b["meta_b"]), meta)


def test_criterion_weight_is_the_tuned_kernel_and_bad_arguments_are_refused():
    I, J, N, M = 256, 256, 2, 4
    W, S, B, perm = _case(I, J, N, M, 5)
    b1, b2 = bm.alloc_layer_buffers(1, I, J, 1), bm.alloc_layer_buffers(1, I, J, 1)
    Wd, pd = dev(W), dev(perm)
    bitsf = dev(O.pack_bits(B).view(np.int32))
    bm.bimask_bwd_mask(Wd, bitsf, pd, I, J, N, M, b1["maskbits_b"], b1["vals_b"], b1["meta_b"], b1["hw_meta_b"])
    bm.bimask_bwd_mask_criterion(Wd, None, bitsf, pd, I, J, N, M, bm.CRIT_WEIGHT, 0, b2["maskbits_b"], b2["vals_b"],
                                 b2["meta_b"], b2["hw_meta_b"])
    # score criterion with S = W must give Eq. 11 as well, through the generic kernel
    b3 = bm.alloc_layer_buffers(1, I, J, 1)
    bm.bimask_bwd_mask_criterion(Wd, Wd, bitsf, pd, I, J, N, M, bm.CRIT_SCORE, 0, b3["maskbits_b"], b3["vals_b"],
                                 b3["meta_b"], b3["hw_meta_b"])
    torch.cuda.synchronize()
    for k in ("maskbits_b", "vals_b", "meta_b", "hw_meta_b"):
        assert torch.equal(b1[k].view(torch.uint8), b2[k].view(torch.uint8)), k
        assert torch.equal(b1[k].view(torch.uint8), b3[k].view(torch.uint8)), k
    n0 = bm.bimask_launch_count()
    for crit, Sarg in ((4, None), (-1, None), (1, None)):
        with pytest.raises(bm.BimaskError) as e:
            bm.bimask_bwd_mask_criterion(Wd, Sarg, bitsf, pd, I, J, N, M, crit, 0, b2["maskbits_b"], b2["vals_b"],
                                         b2["meta_b"], b2["hw_meta_b"])
        assert e.value.code == -1
    assert bm.bimask_launch_count() == n0


def test_random_and_multinomial_statistics_at_scale():
    """On a large i.i.d. layer: the random criterion keeps every competitor of a crowded block with
    the same frequency; the multinomial one prefers large magnitudes but, unlike Eq. 11, not always."""
    I, J, N, M = 2048, 1024, 2, 4
    rng = np.random.default_rng(77)
    W = rng.standard_normal((I, J)).astype(np.float32)
    B = O.forward_mask(W, N, M)
    perm = rng.permutation(I).astype(np.int32)
    Wd, pd = dev(W), dev(perm)
    bitsf = dev(O.pack_bits(B).view(np.int32))
    out = {}
    for crit in (0, 2, 3):
        b = bm.alloc_layer_buffers(1, I, J, 1)
        bm.bimask_bwd_mask_criterion(Wd, None, bitsf, pd, I, J, N, M, crit, 9, b["maskbits_b"], b["vals_b"], b["meta_b"],
                                     b["hw_meta_b"])
        torch.cuda.synchronize()
        out[crit] = O.unpack_bits(u32(b["maskbits_b"]), J)
    Bp = B[perm]
    comp = Bp.reshape(I // M, M, J).sum(axis=1)
    crowded = np.repeat(comp > N, M, axis=0).reshape(I, J) & Bp            # competitors of blocks that must choose
    a = np.abs(W[perm])
    mean_kept = {c: float(a[out[c] & crowded].mean()) for c in out}
    mean_all = float(a[crowded].mean())
    assert mean_kept[0] > mean_kept[2] > mean_all * 1.02                   # Eq. 11 > multinomial > no preference
    assert abs(mean_kept[3] - mean_all) < 0.01 * mean_all                  # random: no preference
    for c in out:
        assert not (out[c] & ~Bp).any()
        assert np.array_equal(out[c].reshape(I // M, M, J).sum(axis=1), np.minimum(comp, N))


# ---------------------------------------------------------------------------------------------
# Greedy refinement of the permutation (bimask_perm_refine)
# ---------------------------------------------------------------------------------------------
def _refine_gpu(B, perm, N, M, rounds, seed):
    I, J = B.shape
    bits = dev(O.pack_bits(B).view(np.int32))
    p = dev(np.asarray(perm, dtype=np.int32))
    cnt = torch.zeros(1, dtype=torch.int64, device="cuda")
    nbytes = bm.bimask_refine_workspace_bytes(I, M, rounds)
    ws = torch.empty(max(nbytes, 16), dtype=torch.uint8, device="cuda")
    bm.bimask_perm_refine(bits, I, J, N, M, rounds, seed, p, cnt, ws, ws.numel())
    torch.cuda.synchronize()
    return p.cpu().numpy(), int(cnt.item())


@pytest.mark.parametrize("I,J,N,M,rounds", [(256, 256, 2, 4, 8), (128, 512, 1, 4, 5), (256, 128, 2, 8, 6),
                                            (128, 64, 1, 16, 4), (64, 96, 4, 8, 3), (96, 160, 2, 4, 7), (64, 64, 2, 4, 0)])
def test_perm_refine_bit_exact(I, J, N, M, rounds):
    rng = np.random.default_rng(I + J + N + M)
    W = rng.standard_normal((I, J)).astype(np.float32)
    B = O.forward_mask(W, N, M)
    perm0 = rng.permutation(I).astype(np.int32)
    seed = 1000 + rounds
    got, cnt = _refine_gpu(B, perm0, N, M, rounds, seed)
    ref, ref_cnt = O.refine_perm(B, perm0, N, M, rounds, seed)
    assert np.array_equal(got, ref)
    assert cnt == ref_cnt
    assert cnt >= O.eligible_blocks(B, perm0, N, M)


def test_perm_refine_at_scale_properties():
    """Too large for the oracle's loops: the result is a permutation, the count equals an independent score of
    the result, grows with the number of rounds and beats the best of the random candidates."""
    I, J, N, M, P = 4096, 2048, 2, 4, 64
    rng = np.random.default_rng(4)
    W = rng.standard_normal((I, J)).astype(np.float32)
    B = O.forward_mask(W, N, M)
    bits = dev(O.pack_bits(B).view(np.int32))
    b = bm.alloc_layer_buffers(1, I, J, P)
    bm.bimask_perm_search(bits, I, J, N, M, P, 7, None, b["perm"], b["best_idx"], b["counts"], b["ws"], b["ws"].numel())
    torch.cuda.synchronize()
    start = b["perm"].cpu().numpy()
    best_random = int(b["counts"].max().item())
    prev = best_random
    for rounds in (4, 16, 48):
        got, cnt = _refine_gpu(B, start, N, M, rounds, 3)
        assert np.array_equal(np.sort(got), np.arange(I))
        assert cnt == O.eligible_blocks(B, got, N, M)
        assert cnt > prev
        prev = cnt
    total = (I // M) * J
    assert best_random / total < 0.70 and prev / total > best_random / total + 0.005


def test_perm_refine_rejects_bad_arguments():
    bits = torch.zeros(64, 2, dtype=torch.int32, device="cuda")
    p = torch.arange(64, dtype=torch.int32, device="cuda")
    ws = torch.empty(1 << 16, dtype=torch.uint8, device="cuda")
    n0 = bm.bimask_launch_count()
    for kw in (dict(rounds=-1), dict(N=3), dict(ws_bytes=8), dict(M=32)):
        a = dict(I=64, J=64, N=2, M=4, rounds=2, ws_bytes=ws.numel())
        a.update(kw)
        with pytest.raises(bm.BimaskError):
            bm.bimask_perm_refine(bits, a["I"], a["J"], a["N"], a["M"], a["rounds"], 1, p, None, ws, a["ws_bytes"])
    assert bm.bimask_launch_count() == n0
