"""GPU parity for the optimizer update fused with the next forward mask, and for whole iterations
of Algorithm 1 with its Delta-T schedule (bimask_sgd_fwd_mask, bimask_train_step).

The update is float32 in a fixed operation order on both sides, so weights, momentum and every
integer result are compared bit for bit.  The multi-iteration test uses small-integer activations:
their products and sums are exact in float32, so the weight gradient -- and with it the whole
trajectory of weights, masks and permutations -- has one correct value."""
import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from tests.gpu_util import bits_dev, dev, rel_err, u16, u32

pytestmark = pytest.mark.gpu


def _planted(I, J, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((I, J)) * 0.05).astype(np.float32)
    dW = rng.standard_normal((I, J)).astype(np.float32)
    mom = rng.standard_normal((I, J)).astype(np.float32)
    # ties after the update, zeros of both signs, gradients that cancel the weight exactly
    W[0, :8] = [0.5, 0.5, -0.5, 0.5, 0.0, -0.0, 0.0, -0.0]
    dW[0, :8] = 0.0
    mom[0, :8] = 0.0
    W[1, :4] = [-0.0, 1.0, -0.0, 2.0]
    dW[1, :4] = [-0.0, 0.0, -0.0, 0.0]
    mom[1, :4] = [-0.0, 0.0, 0.0, 0.0]
    # (non-finite weights are outside the update's contract: NaN payloads differ between processors)
    return W, dW, mom


@pytest.mark.parametrize("I,J,N,M", [(256, 256, 2, 4), (128, 384, 1, 4), (96, 160, 2, 4), (64, 64, 2, 8),
                                     (64, 128, 1, 16), (64, 64, 4, 8)])
@pytest.mark.parametrize("use_mom", [True, False])
def test_sgd_fwd_mask_bit_exact(I, J, N, M, use_mom):
    W, dW, mom = _planted(I, J, 7 + I + J)
    lr, mu, wd = 0.05, (0.9 if use_mom else 0.0), 5e-4
    pack = N <= 2
    b = bm.alloc_layer_buffers(1, I, J, 1)
    Wd, dWd = dev(W), dev(dW)
    momd = dev(mom) if use_mom else None
    bm.bimask_sgd_fwd_mask(Wd, dWd, momd, I, J, N, M, lr, mu, wd, b["maskbits_f"],
                           b["vals_f"] if pack else None, b["meta_f"] if pack else None,
                           b["hw_meta_f"] if pack else None)
    torch.cuda.synchronize()
    W_ref, mom_ref = O.sgd_update(W, dW, mom if use_mom else np.zeros_like(W), lr, mu, wd)
    assert np.array_equal(Wd.cpu().numpy().view(np.uint32), W_ref.view(np.uint32))
    if use_mom:
        assert np.array_equal(momd.cpu().numpy().view(np.uint32), mom_ref.view(np.uint32))
    B = O.forward_mask(W_ref, N, M)
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(B))
    if pack:
        _, vals, meta = O.forward_operand(W_ref, B)
        assert np.array_equal(u16(b["vals_f"]), vals)
        assert np.array_equal(u32(b["meta_f"]), meta)
        # the metadata image must be the one the plain mask call writes for the same weights
        b2 = bm.alloc_layer_buffers(1, I, J, 1)
        bm.bimask_fwd_mask(Wd, I, J, N, M, b2["maskbits_f"], b2["vals_f"], b2["meta_f"], b2["hw_meta_f"])
        torch.cuda.synchronize()
        assert torch.equal(b["hw_meta_f"], b2["hw_meta_f"])


def test_sgd_fwd_mask_at_config5_size_on_samples():
    I, J, N, M = 16384, 4096, 2, 4
    rng = np.random.default_rng(9)
    W = (rng.standard_normal((I, J)) * 0.02).astype(np.float32)
    dW = rng.standard_normal((I, J)).astype(np.float32)
    mom = rng.standard_normal((I, J)).astype(np.float32)
    b = bm.alloc_layer_buffers(1, I, J, 1)
    Wd, dWd, momd = dev(W), dev(dW), dev(mom)
    bm.bimask_sgd_fwd_mask(Wd, dWd, momd, I, J, N, M, 0.1, 0.9, 1e-4, b["maskbits_f"], b["vals_f"], b["meta_f"],
                           b["hw_meta_f"])
    torch.cuda.synchronize()
    W_ref, mom_ref = O.sgd_update(W, dW, mom, 0.1, 0.9, 1e-4)
    assert np.array_equal(Wd.cpu().numpy().view(np.uint32), W_ref.view(np.uint32))
    assert np.array_equal(momd.cpu().numpy().view(np.uint32), mom_ref.view(np.uint32))
    rows = np.sort(rng.choice(I, size=192, replace=False))
    rows = np.unique(np.concatenate([rows, [0, 127, 128, I - 1]]))
    B = O.forward_mask(W_ref[rows], N, M)
    assert np.array_equal(u32(b["maskbits_f"])[rows], O.pack_bits(B))
    vals, meta = O.pack_2to4_fast(W_ref[rows], B)
    assert np.array_equal(u16(b["vals_f"])[rows], vals)
    assert np.array_equal(u32(b["meta_f"])[rows], meta)


@pytest.mark.parametrize("I,J,T,N,M,P,dT", [(256, 256, 64, 2, 4, 8, 2), (128, 384, 96, 1, 4, 6, 3),
                                            (96, 160, 40, 2, 4, 5, 2), (128, 128, 64, 2, 8, 6, 2),
                                            (128, 256, 64, 4, 8, 6, 2),
                                            (256, 384, 6000, 2, 4, 6, 2)])     # above a gigaflop: side streams
def test_train_step_trajectory_bit_exact(I, J, T, N, M, P, dT):
    iters, seed = 5, 77
    lr, mu, wd = 2.0 ** -9, 0.5, 2.0 ** -7
    rng = np.random.default_rng(I + J + T)
    W0 = (rng.standard_normal((I, J)) * 0.05).astype(np.float32)
    X = [O.bf16_bits(rng.integers(-3, 4, size=(T, J)).astype(np.float32)) for _ in range(iters)]
    dY = [O.bf16_bits(rng.integers(-3, 4, size=(T, I)).astype(np.float32)) for _ in range(iters)]
    hist, W_fin, mom_fin, sparse_fin = O.train_steps(W0, X, dY, N, M, P, seed, dT, iters, lr, mu, wd)

    pack = N <= 2                      # 4:8 runs on dense masked operands
    b = bm.alloc_layer_buffers(T, I, J, P, dense=not pack)
    b["W"] = dev(W0)
    mom = torch.zeros(I, J, dtype=torch.float32, device="cuda")
    for t in range(1, iters + 1):
        b["X"], b["dY"] = bits_dev(X[t - 1]), bits_dev(dY[t - 1])
        largs = bm.make_layer_args(T, I, J, N, M, P, seed, False, b)
        targs = bm.make_train_args(largs, mom, lr, mu, wd, t, dT, premasked=(t > 1))
        W_seen = b["W"].cpu().numpy().copy()
        bm.bimask_train_step(targs)
        torch.cuda.synchronize()
        h = hist[t - 1]
        assert int(b["status_word"].item()) == 0
        assert np.array_equal(W_seen.view(np.uint32), h["W"].view(np.uint32)), t
        assert np.array_equal(b["perm"].cpu().numpy(), h["perm"]), t
        if h["searched"]:
            assert int(b["best_idx"].item()) == h["best_idx"]
            assert np.array_equal(b["counts"].cpu().numpy(), h["counts"])
        assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(h["Bbar_p"])), t
        if pack:
            assert np.array_equal(u16(b["vals_b"]), h["vals_b"]), t
            assert np.array_equal(u32(b["meta_b"]), h["meta_b"]), t
        else:
            assert np.array_equal(u16(b["vals_b"]), O.dense_backward_operand(h["W"], h["Bbar_p"], h["perm"])), t
        assert np.array_equal(b["dW"].cpu().numpy(), h["dW"].astype(np.float32)), t     # exact: integer data
        assert rel_err(b["Y"].float().cpu().numpy(), h["Y"]) <= 2e-2
        assert rel_err(b["dX"].float().cpu().numpy(), h["dX"]) <= 2e-2
    assert np.array_equal(b["W"].cpu().numpy().view(np.uint32), W_fin.view(np.uint32))
    assert np.array_equal(mom.cpu().numpy().view(np.uint32), mom_fin.view(np.uint32))
    # the forward operand left behind is B . W of the final weights: the algorithm's return value
    B_fin = O.forward_mask(W_fin, N, M)
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(B_fin))
    if pack:
        _, vals, meta = O.forward_operand(W_fin, B_fin)
        assert np.array_equal(u16(b["vals_f"]), vals)
        assert np.array_equal(u32(b["meta_f"]), meta)
    else:
        vals = O.dense_operand(W_fin, B_fin)
        assert np.array_equal(u16(b["vals_f"]), vals)
        assert np.array_equal(O.bf16_to_f64(vals), O.bf16_round(sparse_fin))
    assert np.count_nonzero(O.bf16_to_f64(vals)) == np.count_nonzero(O.bf16_round(sparse_fin))


def test_train_step_rejects_bad_arguments():
    I, J, T, P = 128, 128, 32, 4
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"] = torch.zeros(I, J, device="cuda")
    b["X"] = torch.zeros(T, J, dtype=torch.bfloat16, device="cuda")
    b["dY"] = torch.zeros(T, I, dtype=torch.bfloat16, device="cuda")
    largs = bm.make_layer_args(T, I, J, 2, 4, P, 1, False, b)
    n0 = bm.bimask_launch_count()
    for kw in (dict(t=0, delta_t=1), dict(t=1, delta_t=0), dict(t=1, delta_t=1, lr=float("nan"))):
        targs = bm.make_train_args(largs, None, kw.get("lr", 0.1), 0.0, 0.0, kw["t"], kw["delta_t"], False)
        with pytest.raises(bm.BimaskError) as e:
            bm.bimask_train_step(targs)
        assert e.value.code == -1
    assert bm.bimask_launch_count() == n0
