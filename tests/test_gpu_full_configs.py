"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times
(bimask_layer_step on every layer of a config).

Configs 2, 3 and 4 (ResNet-50-shaped convolutions at 2:4 and 1:4, DeiT-small linears) are small
enough for the oracle to recompute every output in full.  Config 5 (16384 x 4096 and 4096 x 16384 at
8192 tokens) is checked on samples the oracle computes one by one: whole rows of the forward
operand, whole permuted row-blocks of the backward operand, the eligible-block counts of a sample
of candidates (plus the property that the chosen one is the first maximiser of all counts), and
whole rows / columns of the three products including the rows and columns next to tile borders."""
import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from paper_2302_06058_b200 import inputs
from tests.gpu_util import rel_err, run_layer_step, u16, u32

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _layers(cfg_id):
    return [(cfg_id, li) for li in range(len(inputs.CONFIGS[cfg_id].layers))]


@pytest.mark.parametrize("cfg_id,li", _layers(2) + _layers(3) + _layers(4))
def test_full_layer_against_full_oracle(cfg_id, li):
    cfg = inputs.CONFIGS[cfg_id]
    W, X, dY = inputs.make_layer(cfg_id, li)
    seed = inputs.perm_seed(cfg_id)
    b = run_layer_step(W, X, dY, cfg.N, cfg.M, cfg.P, seed, do_search=True)
    ref = O.layer_step(W, X, dY, cfg.N, cfg.M, cfg.P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(u32(b["meta_f"]), ref["meta_f"])
    assert np.array_equal(u16(b["vals_f"]), ref["vals_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert int(b["best_idx"].item()) == ref["best_idx"]
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u32(b["meta_b"]), ref["meta_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy(), ref["Y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL


def _border_indices(n, tile, rng, extra):
    idx = {0, n - 1}
    for t in range(tile, n, tile):
        idx.update((t - 1, t))
    picks = sorted(idx)
    if len(picks) > 24:
        picks = list(rng.choice(picks, size=24, replace=False))
    picks += list(rng.integers(0, n, size=extra))
    return np.array(sorted(set(int(i) for i in picks)), dtype=np.int64)


@pytest.mark.parametrize("li", [0, 1])
def test_config5_layer_on_samples(li):
    cfg_id = 5
    cfg = inputs.CONFIGS[cfg_id]
    L = cfg.layers[li]
    I, J, T, N, M, P = L.I, L.J, L.T, cfg.N, cfg.M, cfg.P
    W, X, dY = inputs.make_layer(cfg_id, li)
    seed = inputs.perm_seed(cfg_id)
    b = run_layer_step(W, X, dY, N, M, P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    rng = np.random.default_rng(50 + li)

    # ---- forward mask, row chunks (the mask is row-local, so chunks reproduce the full result)
    B = np.empty((I, J), dtype=bool)
    for r0 in range(0, I, 1024):
        B[r0:r0 + 1024] = O.forward_mask(W[r0:r0 + 1024], N, M)
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(B))
    rows = np.sort(rng.choice(I, size=256, replace=False))
    vals, meta = O.pack_2to4_fast(W[rows], B[rows])
    assert np.array_equal(u16(b["vals_f"])[rows], vals)
    assert np.array_equal(u32(b["meta_f"])[rows], meta)

    # ---- search: counts of a sample of candidates; the pick is the first maximiser of all counts
    cands = O.candidates(seed, P, I)
    got_counts = b["counts"].cpu().numpy()
    best = int(b["best_idx"].item())
    for c in sorted({0, 1, P // 2, P - 1, best} | set(int(x) for x in rng.integers(0, P, size=3))):
        assert got_counts[c] == O.eligible_blocks(B, cands[c], N, M), c
    assert best == int(np.argmax(got_counts))
    perm = b["perm"].cpu().numpy()
    assert np.array_equal(perm, cands[best])
    # closed form: for i.i.d. weights 11/16 of the blocks are eligible, whatever the row order
    nblocks = (I // M) * J
    assert abs(got_counts.mean() / nblocks - 11 / 16) < 1e-3

    # ---- backward mask: the full mask in chunks of permuted rows (column-block local given perm),
    #      the transposed packed operand on sampled 32-row slabs (one metadata word each)
    got_bits_b = u32(b["maskbits_b"])
    got_vals_b = u16(b["vals_b"])
    got_meta_b = u32(b["meta_b"])
    Bbar_all = np.empty((I, J), dtype=bool)
    for r0 in range(0, I, 1024):
        prow = perm[r0:r0 + 1024]
        Bbar_all[r0:r0 + 1024] = O.backward_mask(W[prow], B[prow], np.arange(len(prow)), N, M)
    assert np.array_equal(got_bits_b, O.pack_bits(Bbar_all))
    for k0 in sorted(set(int(x) for x in rng.integers(0, I // 32, size=6)) | {0, I // 32 - 1}):
        prow = perm[32 * k0: 32 * k0 + 32]
        Bb = Bbar_all[32 * k0: 32 * k0 + 32]
        v, m = O.pack_2to4_fast(np.ascontiguousarray(W[prow].T), np.ascontiguousarray(Bb.T))
        assert np.array_equal(got_vals_b[:, 16 * k0: 16 * k0 + 16], v)
        assert np.array_equal(got_meta_b[:, k0], m[:, 0])
    assert not (Bbar_all & ~B[perm]).any()
    assert int(Bbar_all.reshape(I // M, M, J).sum(axis=1).max()) <= N

    # ---- products on whole sampled rows and columns (tile borders included)
    Wr = O.bf16_round(W)
    Xf = O.bf16_to_f64(X)
    dYf = O.bf16_to_f64(dY)
    Y = b["Y"].float().cpu().numpy()
    dX = b["dX"].float().cpu().numpy()
    dW = b["dW"].cpu().numpy()
    ts = _border_indices(T, 256, rng, 16)
    is_ = _border_indices(I, 128, rng, 16)
    js = _border_indices(J, 128, rng, 16)
    Wf = Wr * B
    ref = Xf[ts] @ Wf.T                                        # Y[ts, :]
    assert rel_err(Y[ts], ref) <= TOL
    ref = Xf @ Wf[is_].T                                       # Y[:, is]
    assert rel_err(Y[:, is_], ref) <= TOL
    Mb = np.zeros((I, J), dtype=bool)
    Mb[perm] = Bbar_all                                        # the oracle's backward mask, original row order
    Wb = Wr * Mb
    ref = dYf[ts] @ Wb                                         # dX[ts, :]
    assert rel_err(dX[ts], ref) <= TOL
    ref = dYf @ Wb[:, js]                                      # dX[:, js]
    assert rel_err(dX[:, js], ref) <= TOL
    ref = dYf[:, is_].T @ Xf                                   # dW[is, :]
    assert rel_err(dW[is_], ref) <= TOL
    ref = dYf.T @ Xf[:, js]                                    # dW[:, js]
    assert rel_err(dW[:, js], ref) <= TOL


@pytest.mark.parametrize("I,J,T", [(256, 64, 100352), (64, 256, 100352), (2048, 512, 1568), (512, 2048, 1568)])
def test_resnet_bottleneck_1x1_shapes(I, J, T):
    """The 1x1 convolutions of ResNet-50's bottleneck blocks (c x 4c and 4c x c at the same pixel counts as
    config 2) are plain linear layers on the NHWC activations: narrow reduction or narrow output, very many tokens."""
    N, M, P, seed = 2, 4, 32, 44
    W = inputs.make_weight(I, J, 600 + I)
    X = inputs.make_activation(T, J, 601)
    dY = inputs.make_activation(T, I, 602)
    b = run_layer_step(W, X, dY, N, M, P, seed, do_search=True)
    ref = O.layer_step(W, X, dY, N, M, P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(u16(b["vals_f"]), ref["vals_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy(), ref["Y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL
