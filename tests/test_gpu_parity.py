"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs.  Integer outputs (mask bits, packed values and codes, counts, the chosen
permutation) must match bit for bit; products within max |y - ref| / max(|ref|, rms(ref)) <= 2e-2
(bf16 inputs, fp32 accumulation, bf16 outputs for Y and dX)."""
import itertools

import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from paper_2302_06058_b200 import inputs
from tests.gpu_util import bits_dev, dev, rel_err, run_fwd_mask, run_layer_step, u16, u32

pytestmark = pytest.mark.gpu
TOL = 2e-2


def special_weights(I, J, seed):
    """Normal weights with planted ties, zeros, negative zeros, denormals, inf and NaN."""
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((I, J)).astype(np.float32)
    W[rng.random((I, J)) < 0.15] = 0.0
    W[rng.random((I, J)) < 0.05] = -0.0
    t = rng.random((I, J)) < 0.2
    W[t] = np.round(W[t] * 2) / 2                       # many equal magnitudes
    W[0, :8] = [np.inf, -np.inf, 1.0, np.nan, 1e-41, -1e-41, 3.0, -3.0]
    return W


@pytest.mark.parametrize("I,J,N", [(256, 256, 2), (32, 32, 2), (64, 576, 2), (96, 160, 1), (512, 4608, 1),
                                   (1152, 384, 2), (2048, 1056, 2)])
def test_fwd_mask_bit_exact(I, J, N):
    W = special_weights(I, J, I + J + N) if I < 1000 else inputs.make_weight(I, J, 5)
    _, b = run_fwd_mask(W, N)
    B = O.forward_mask(W, N, 4)
    bits, vals, meta = O.forward_operand(W, B)
    assert np.array_equal(u32(b["maskbits_f"]), bits)
    assert np.array_equal(u32(b["meta_f"]), meta)
    assert np.array_equal(u16(b["vals_f"]), vals)


@pytest.mark.parametrize("I,J,N", [(256, 256, 2), (32, 32, 1), (64, 576, 2), (96, 160, 1), (512, 1184, 2),
                                   (1152, 384, 2)])
def test_bwd_mask_bit_exact(I, J, N):
    W = special_weights(I, J, 3 * I + J + N)
    Wd, b = run_fwd_mask(W, N)
    perm = np.random.default_rng(I).permutation(I).astype(np.int32)
    pd = dev(perm)
    bm.bimask_bwd_mask(Wd, b["maskbits_f"], pd, I, J, N, 4, b["maskbits_b"], b["vals_b"], b["meta_b"], b["hw_meta_b"])
    torch.cuda.synchronize()
    B = O.forward_mask(W, N, 4)
    Bbar = O.backward_mask(W, B, perm, N, 4)
    bits, vals, meta = O.backward_operand(W, Bbar, perm)
    assert np.array_equal(u32(b["maskbits_b"]), bits)
    assert np.array_equal(u32(b["meta_b"]), meta)
    assert np.array_equal(u16(b["vals_b"]), vals)


@pytest.mark.parametrize("I,P,cap", [(20000, 3, 0), (20000, 3, 700), (40000, 2, 3000), (4096, 4, 300), (8192, 2, 64),
                                     (16384, 5, 0), (12288, 3, 0), (100, 7, 0), (100, 7, 16)])
def test_candidate_generator_alone_and_with_a_forced_small_part_buffer(I, P, cap):
    """The generator's result must not depend on how many keys a sorting pass may hold: with a small capacity the
    part-wise kernel sorts a part in several passes (the path a part takes if it ever draws more keys than its
    buffer holds) and still produces the oracle's candidates."""
    seed = 1234 + I
    cands = torch.full((P, I), -7, dtype=torch.int32, device="cuda")
    bm.bimask_debug_gen_candidates(seed, P, I, cap, cands)
    torch.cuda.synchronize()
    assert np.array_equal(cands.cpu().numpy(), O.candidates(seed, P, I))


@pytest.mark.parametrize("I,J,N,P", [(256, 256, 2, 8), (64, 576, 2, 32), (512, 4608, 1, 64), (1152, 384, 2, 32),
                                     (100, 96, 2, 5), (16384, 64, 2, 3), (40000, 32, 2, 2),
                                     (128, 128, 2, 1), (96, 64, 1, 300), (2048, 2048, 2, 130)])
def test_perm_search_generated(I, J, N, P):
    W = inputs.make_weight(I, J, I + P)
    B = O.forward_mask(W, N, 4)
    bits = dev(O.pack_bits(B).view(np.int32))
    ws_bytes = bm.bimask_workspace_bytes(1, I, J, P)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    best_perm = torch.empty(I, dtype=torch.int32, device="cuda")
    best_idx = torch.empty(1, dtype=torch.int32, device="cuda")
    counts = torch.empty(P, dtype=torch.int64, device="cuda")
    seed = 42 + I
    bm.bimask_perm_search(bits, I, J, N, 4, P, seed, None, best_perm, best_idx, counts, ws, ws_bytes)
    torch.cuda.synchronize()
    cands = O.candidates(seed, P, I)
    best, perm, cnt = O.perm_search(B, cands, N, 4)
    got_cands = ws[: P * I * 4].view(torch.int32).view(P, I).cpu().numpy()
    assert np.array_equal(got_cands, cands)
    assert np.array_equal(counts.cpu().numpy(), cnt)
    assert int(best_idx.item()) == best
    assert np.array_equal(best_perm.cpu().numpy(), perm)
    ok = torch.zeros(1, dtype=torch.int32, device="cuda")
    scratch = torch.empty(P * I, dtype=torch.uint8, device="cuda")
    bm.bimask_check_perms(ws[: P * I * 4].view(torch.int32), P, I, ok, scratch, P * I)
    assert int(ok.item()) == 1


def test_perm_search_all_permutations_of_8_rows():
    """All 8! explicit candidates on the hand-worked 8 x 8 example (tiled to 32 columns, so every
    count is four times the 8 x 8 one): counts and the first maximiser must match."""
    from tests.test_oracle_pins import _read_example, brute_count
    W8, B8, _ = _read_example()
    B = np.tile(B8, (1, 4))
    allp = np.array(list(itertools.permutations(range(8))), dtype=np.int32)
    P = allp.shape[0]
    bits = dev(O.pack_bits(B).view(np.int32))
    best_perm = torch.empty(8, dtype=torch.int32, device="cuda")
    best_idx = torch.empty(1, dtype=torch.int32, device="cuda")
    counts = torch.empty(P, dtype=torch.int64, device="cuda")
    bm.bimask_perm_search(bits, 8, 32, 2, 4, P, 0, dev(allp), best_perm, best_idx, counts, None, 0)
    torch.cuda.synchronize()
    ref8 = np.array([brute_count(B8, p, 2, 4) for p in allp])
    got = counts.cpu().numpy()
    assert np.array_equal(got, 4 * ref8)
    first = int(np.nonzero(ref8 == 16)[0][0])
    assert int(best_idx.item()) == first
    assert np.array_equal(best_perm.cpu().numpy(), allp[first])
    best, perm, cnt = O.perm_search(B, allp, 2, 4)
    assert best == first and np.array_equal(cnt, got)


def test_planted_permutation_wins():
    I, J, N = 256, 512, 2
    W, Q = inputs.planted_transposable(I, J, N, 4, 77)
    rng = np.random.default_rng(1)
    cands = np.stack([rng.permutation(I) for _ in range(6)] + [Q] + [rng.permutation(I) for _ in range(4)]).astype(np.int32)
    X = inputs.make_activation(64, J, 1)
    dY = inputs.make_activation(64, I, 2)
    b = run_layer_step(W, X, dY, N, 4, cands.shape[0], 0, do_search=True, cands=cands)
    assert int(b["best_idx"].item()) == 6
    assert int(b["counts"][6].item()) == (I // 4) * J
    assert np.array_equal(b["perm"].cpu().numpy(), Q)
    B = O.forward_mask(W, N, 4)
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(B[Q]))        # B-bar == B[perm]
    exact = O.dense_dgrad(dY, W, B)                                         # Eq. 5
    got = b["dX"].float().cpu().numpy()
    assert rel_err(got, exact) <= TOL


GEMM_SHAPES = [  # (I, J, T, N)
    (256, 256, 128, 2),      # config 1
    (128, 128, 128, 2),      # exactly one tile
    (64, 576, 300, 2),       # rows < tile, ragged reduction (576 = 4.5 x 128), ragged tokens
    (384, 384, 129, 1),      # 1:4 in the 2:4 container, T = tile + 1
    (160, 96, 1, 2),         # a single token
    (512, 1184, 1568, 2),    # several tiles each way with ragged tails
]


@pytest.mark.parametrize("I,J,T,N", GEMM_SHAPES)
def test_layer_step_parity(I, J, T, N):
    W = inputs.make_weight(I, J, 11 * I + J)
    X = inputs.make_activation(T, J, 5 * I + T)
    dY = inputs.make_activation(T, I, 7 * J + T)
    P, seed = 6, 1234 + I
    b = run_layer_step(W, X, dY, N, 4, P, seed, do_search=True)
    ref = O.layer_step(W, X, dY, N, 4, P, seed, do_search=True)
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


def test_metadata_round_trip_through_the_tensor_core():
    """Multiply the packed forward operand by an identity activation: the product must be the
    masked, bf16-rounded weight itself, exactly (pins the opaque metadata order)."""
    I = J = T = 256
    W = inputs.make_weight(I, J, 99)
    Wd, b = run_fwd_mask(W, 2)
    X = torch.eye(J, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty(T, I, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    bm.bimask_spmm_fwd(X, b["vals_f"], b["hw_meta_f"], T, I, J, Y, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    B = O.forward_mask(W, 2, 4)
    expect = (O.bf16_round(W) * B).T                  # Y[t, i] = (B*W)[i, t]
    assert np.array_equal(Y.float().cpu().numpy().astype(np.float64), expect)


def _tmem_image(meta, rows, kwords):
    """The tensor-memory image of the index codes, rebuilt from the canonical code words by the layout the header
    documents: one 2048-byte block per (128 rows, 4 code words); image lane L = m0 + 8 h + 16 m2 (m0 < 8, h < 2,
    m2 < 8) and column c hold, for code word 4 kt + c, half h (low / high 16 bits) of row m0 + 16 m2 in the low 16
    bits and of row m0 + 8 + 16 m2 in the high 16 bits; entries past the matrix hold the code 0x4 in every nibble."""
    tm, tk = (rows + 127) // 128, (kwords + 3) // 4
    full = np.full((tm * 128, tk * 4), 0x44444444, dtype=np.uint64)
    full[:rows, :kwords] = meta.astype(np.uint64)
    img = np.zeros((tm, tk, 128, 4), dtype=np.uint32)
    for L in range(128):
        m0, h, m2 = L & 7, (L >> 3) & 1, L >> 4
        lo_rows = np.arange(tm) * 128 + m0 + 16 * m2
        lo = (full[lo_rows] >> (16 * h)) & 0xFFFF                 # [tm, tk * 4]
        hi = (full[lo_rows + 8] >> (16 * h)) & 0xFFFF
        img[:, :, L, :] = (lo | (hi << 16)).astype(np.uint32).reshape(tm, tk, 4)
    return img.reshape(-1)


@pytest.mark.parametrize("I,J,N", [(256, 256, 2), (64, 576, 2), (96, 160, 1), (512, 1184, 2), (1152, 384, 2), (32, 32, 2)])
def test_metadata_images_of_both_operands_padding_included(I, J, N):
    """The mask kernels write the tensor-core order of the index codes themselves, on shapes with and without
    padding: compare both images, word for word, with a re-ordering of the (oracle-checked) canonical code words."""
    W = special_weights(I, J, 7 * I + J) if I < 1000 else inputs.make_weight(I, J, 6)
    Wd, b = run_fwd_mask(W, N)
    b["hw_meta_f"].fill_(255)                             # stale contents must not survive anywhere, padding included
    bm.bimask_fwd_mask(Wd, I, J, N, 4, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    perm = np.random.default_rng(J).permutation(I).astype(np.int32)
    b["hw_meta_b"].fill_(255)
    bm.bimask_bwd_mask(Wd, b["maskbits_f"], dev(perm), I, J, N, 4, b["maskbits_b"], b["vals_b"], b["meta_b"], b["hw_meta_b"])
    torch.cuda.synchronize()
    got_f = b["hw_meta_f"].cpu().numpy().view(np.uint32)
    got_b = b["hw_meta_b"].cpu().numpy().view(np.uint32)
    assert np.array_equal(got_f[: ((I + 127) // 128) * ((J // 32 + 3) // 4) * 512], _tmem_image(u32(b["meta_f"]), I, J // 32))
    assert np.array_equal(got_b[: ((J + 127) // 128) * ((I // 32 + 3) // 4) * 512], _tmem_image(u32(b["meta_b"]), J, I // 32))


def test_do_search_zero_uses_given_perm():
    I, J, T = 128, 160, 70
    W = inputs.make_weight(I, J, 3)
    X = inputs.make_activation(T, J, 4)
    dY = inputs.make_activation(T, I, 5)
    perm = np.random.default_rng(9).permutation(I).astype(np.int32)
    b = run_layer_step(W, X, dY, 2, 4, 1, 0, do_search=False, perm=perm)
    ref = O.layer_step(W, X, dY, 2, 4, 1, 0, do_search=False, perm=perm)
    assert np.array_equal(b["perm"].cpu().numpy(), perm)
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL


def test_search_with_the_largest_candidate_count():
    """P = 65535, the documented maximum (one grid row per candidate): counts, winner and permutation against the
    oracle on a matrix small enough for the oracle to score every candidate; one more candidate is refused."""
    I, J, P, seed = 32, 64, 65535, 5
    W = inputs.make_weight(I, J, 17)
    B = O.forward_mask(W, 2, 4)
    bits = dev(O.pack_bits(B).view(np.int32))
    ws_bytes = bm.bimask_workspace_bytes(1, I, J, P)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
    best_perm = torch.empty(I, dtype=torch.int32, device="cuda")
    best_idx = torch.empty(1, dtype=torch.int32, device="cuda")
    counts = torch.empty(P + 1, dtype=torch.int64, device="cuda")
    bm.bimask_perm_search(bits, I, J, 2, 4, P, seed, None, best_perm, best_idx, counts, ws, ws_bytes)
    torch.cuda.synchronize()
    cands = O.candidates(seed, P, I)
    best, perm, cnt = O.perm_search(B, cands, 2, 4)
    assert np.array_equal(counts[:P].cpu().numpy(), cnt)
    assert int(best_idx.item()) == best
    assert np.array_equal(best_perm.cpu().numpy(), perm)
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_perm_search(bits, I, J, 2, 4, P + 1, seed, None, best_perm, best_idx, counts, ws, ws_bytes)
    assert e.value.code == bm.binding.BIMASK_EINVAL


def test_layer_step_at_the_largest_row_count():
    """I = 51200, the documented limit of the layer step (the permutation pass keeps a row of dY in shared memory):
    masks, counts and the permutation bit for bit, the three products within tolerance; four rows more are refused."""
    I, J, T, P, seed = 51200, 64, 96, 2, 11
    W = inputs.make_weight(I, J, 23)
    X = inputs.make_activation(T, J, 24)
    dY = inputs.make_activation(T, I, 25)
    b = run_layer_step(W, X, dY, 2, 4, P, seed, do_search=True)
    ref = O.layer_step(W, X, dY, 2, 4, P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    for n in ("Y", "dX", "dW"):
        assert rel_err(b[n].float().cpu().numpy(), ref[n]) <= TOL, n
    I2 = I + 4
    b2 = bm.alloc_layer_buffers(T, I2, J, P)
    b2["W"] = torch.zeros(I2, J, device="cuda")
    b2["X"] = torch.zeros(T, J, dtype=torch.bfloat16, device="cuda")
    b2["dY"] = torch.zeros(T, I2, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_layer_step(bm.make_layer_args(T, I2, J, 2, 4, P, seed, True, b2))
    assert e.value.code in (bm.binding.BIMASK_EUNSUPPORTED, bm.binding.BIMASK_EINVAL)


def test_error_paths_launch_nothing():
    W = torch.zeros(64, 64, device="cuda")
    b = bm.alloc_layer_buffers(8, 64, 64, 2)
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_fwd_mask(W, 64, 48, 2, 4, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EINVAL
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_fwd_mask(W, 64, 64, 2, 32, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EUNSUPPORTED
    with pytest.raises(bm.BimaskError) as e:     # 4:8 has no 2:4 container: there is no metadata to write
        bm.bimask_fwd_mask(W, 64, 64, 4, 8, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EUNSUPPORTED
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_fwd_mask(W, 64, 64, 3, 4, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EUNSUPPORTED
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_fwd_mask(None, 64, 64, 2, 4, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EINVAL
    with pytest.raises(bm.BimaskError) as e:     # misaligned pointer
        bm.bimask_fwd_mask(W.data_ptr() + 4, 64, 64, 2, 4, b["maskbits_f"], b["vals_f"], b["meta_f"], b["hw_meta_f"])
    assert e.value.code == bm.binding.BIMASK_EINVAL
    with pytest.raises(bm.BimaskError) as e:     # P = 0
        bm.bimask_perm_search(b["maskbits_f"], 64, 64, 2, 4, 0, 1, None, b["perm"], b["best_idx"], b["counts"], b["ws"], 1 << 20)
    assert e.value.code == bm.binding.BIMASK_EINVAL
    with pytest.raises(bm.BimaskError) as e:     # workspace too small
        bm.bimask_perm_search(b["maskbits_f"], 64, 64, 2, 4, 2, 1, None, b["perm"], b["best_idx"], b["counts"], b["ws"], 16)
    assert e.value.code == bm.binding.BIMASK_EINVAL
    assert "workspace" in bm.bimask_last_error()
    torch.cuda.synchronize()


def test_layer_step_host_matches_device_path():
    """The end-to-end entry (host buffers in, host buffers out) gives the same bits as the device
    path and leaves the status word at zero."""
    I, J, T, N, P, seed = 256, 384, 200, 2, 5, 77
    W = inputs.make_weight(I, J, 31)
    X = inputs.make_activation(T, J, 32)
    dY = inputs.make_activation(T, I, 33)
    ref = run_layer_step(W, X, dY, N, 4, P, seed, do_search=True)
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"] = torch.empty(I, J, device="cuda")
    b["X"] = torch.empty(T, J, dtype=torch.bfloat16, device="cuda")
    b["dY"] = torch.empty(T, I, dtype=torch.bfloat16, device="cuda")
    dev_args = bm.make_layer_args(T, I, J, N, 4, P, seed, True, b)
    host = {
        "W": torch.from_numpy(W).pin_memory(),
        "X": torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory(),
        "dY": torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).pin_memory(),
        "Y": torch.empty(T, I, dtype=torch.bfloat16).pin_memory(),
        "dX": torch.empty(T, J, dtype=torch.bfloat16).pin_memory(),
        "dW": torch.empty(I, J, dtype=torch.float32).pin_memory(),
        "perm": torch.empty(I, dtype=torch.int32).pin_memory(),
        "best_idx": torch.empty(1, dtype=torch.int32).pin_memory(),
        "counts": torch.empty(P, dtype=torch.int64).pin_memory(),
        "maskbits_f": torch.empty(I, J // 32, dtype=torch.int32).pin_memory(),
        "maskbits_b": torch.empty(I, J // 32, dtype=torch.int32).pin_memory(),
    }
    hst = torch.full((1,), -9, dtype=torch.int32).pin_memory()
    bm.bimask_layer_step_host(dev_args, bm.make_layer_args(T, I, J, N, 4, P, seed, True, host), hst)
    assert int(hst.item()) == 0
    assert torch.equal(host["Y"], ref["Y"].cpu())
    assert torch.equal(host["dX"], ref["dX"].cpu())
    assert torch.equal(host["dW"], ref["dW"].cpu())
    assert torch.equal(host["perm"], ref["perm"].cpu())
    assert torch.equal(host["counts"], ref["counts"].cpu())
    assert int(host["best_idx"].item()) == int(ref["best_idx"].item())
    assert torch.equal(host["maskbits_f"], ref["maskbits_f"].cpu())
    assert torch.equal(host["maskbits_b"], ref["maskbits_b"].cpu())
    # the non-blocking form: two calls in flight (the second re-uses the same buffers), then one wait
    for name in ("Y", "dX", "dW"):
        host[name].zero_()
    hst.fill_(-9)
    hargs = bm.make_layer_args(T, I, J, N, 4, P, seed, True, host)
    bm.bimask_layer_step_host_async(dev_args, hargs, hst)
    bm.bimask_layer_step_host_async(dev_args, hargs, hst)
    bm.bimask_host_sync()
    assert int(hst.item()) == 0
    assert torch.equal(host["Y"], ref["Y"].cpu())
    assert torch.equal(host["dX"], ref["dX"].cpu())
    assert torch.equal(host["dW"], ref["dW"].cpu())


def test_layer_step_is_deterministic():
    """Two runs on the same inputs give identical bits (no atomics on floating-point data)."""
    I, J, T = 512, 256, 333
    W = inputs.make_weight(I, J, 41)
    X = inputs.make_activation(T, J, 42)
    dY = inputs.make_activation(T, I, 43)
    a = run_layer_step(W, X, dY, 2, 4, 4, 5, do_search=True)
    b = run_layer_step(W, X, dY, 2, 4, 4, 5, do_search=True)
    for name in ("Y", "dX", "dW", "perm", "counts", "maskbits_f", "maskbits_b", "vals_f", "vals_b", "meta_f", "meta_b",
                 "hw_meta_f", "hw_meta_b"):
        assert torch.equal(a[name], b[name]), name


def test_small_layer_with_split_k_weight_gradient():
    """Few output tiles and many tokens: the weight gradient is split along the tokens."""
    I, J, T = 64, 96, 9000
    W = inputs.make_weight(I, J, 51)
    X = inputs.make_activation(T, J, 52)
    dY = inputs.make_activation(T, I, 53)
    b = run_layer_step(W, X, dY, 2, 4, 3, 6, do_search=True)
    ref = O.layer_step(W, X, dY, 2, 4, 3, 6, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL
    assert rel_err(b["Y"].float().cpu().numpy(), ref["Y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL


@pytest.mark.parametrize("I,J,T", [(96, 160, 129), (32, 32, 70), (64, 96, 9000), (160, 288, 1000), (1152, 384, 1500),
                                   (2080, 4128, 530)])
def test_products_write_nothing_outside_their_results(I, J, T):
    """Y, dX and dW leave the kernels as tensor stores of whole boxes that the tensor maps clip at the edge of the
    result: the three results are placed inside larger buffers filled with a sentinel, on ragged shapes in every
    dimension (partial row tiles, partial token chunks, split-K partial sums), and the sentinel must survive around
    them while the results themselves still match."""
    W = inputs.make_weight(I, J, 3 * I + J)
    X = inputs.make_activation(T, J, I + T)
    dY = inputs.make_activation(T, I, J + T)
    P, seed, pad = 3, 99, 4096
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"], b["X"], b["dY"] = dev(W), bits_dev(X), bits_dev(dY)
    guards = {}
    for name, dt, sentinel in (("Y", torch.bfloat16, 7.0), ("dX", torch.bfloat16, 7.0), ("dW", torch.float32, 7.0)):
        n = b[name].numel()
        big = torch.full((n + 2 * pad,), sentinel, dtype=dt, device="cuda")
        guards[name] = big
        b[name] = big[pad:pad + n].view(b[name].shape)
    bm.bimask_layer_step(bm.make_layer_args(T, I, J, 2, 4, P, seed, True, b))
    torch.cuda.synchronize()
    ref = O.layer_step(W, X, dY, 2, 4, P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    for name, big in guards.items():
        assert bool((big[:pad] == 7.0).all()) and bool((big[-pad:] == 7.0).all()), name
        assert rel_err(b[name].float().cpu().numpy(), ref[name]) <= TOL, name


# ---------------------------------------------------------------------------------------------
# The other N:M patterns the paper trains (4:8, 2:8, 1:8, 1:16): masks, search, backward mask bit
# for bit; those that fit the 2:4 container (N <= 2) also run the whole layer step.
# ---------------------------------------------------------------------------------------------
NM_PATTERNS = [(2, 8), (1, 8), (1, 16), (4, 8), (2, 16)]


@pytest.mark.parametrize("N,M", NM_PATTERNS)
@pytest.mark.parametrize("I,J", [(64, 96), (256, 384), (1024, 1056)])
def test_other_patterns_masks_and_search(N, M, I, J):
    W = special_weights(I, J, 7 * I + J + N + M) if I < 1000 else inputs.make_weight(I, J, N + M)
    pack = N <= 2
    Wd = dev(W)
    b = bm.alloc_layer_buffers(1, I, J, 4, dense=not pack)
    opt = (lambda t: t) if pack else (lambda t: None)
    bm.bimask_fwd_mask(Wd, I, J, N, M, b["maskbits_f"], b["vals_f"], opt(b["meta_f"]), opt(b["hw_meta_f"]))
    B = O.forward_mask(W, N, M)
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(B))
    if pack:
        _, vals, meta = O.forward_operand(W, B)
        assert np.array_equal(u32(b["meta_f"]), meta)
        assert np.array_equal(u16(b["vals_f"]), vals)
    else:                                   # no 2:4 form: the dense masked operand
        assert np.array_equal(u16(b["vals_f"]), O.dense_operand(W, B))
        before = b["maskbits_f"].clone()
        bm.bimask_fwd_mask(Wd, I, J, N, M, b["maskbits_f"], None, None, None)        # mask bits only
        assert torch.equal(before, b["maskbits_f"])
    # search
    P, seed = 4, 99 + M
    ws_bytes = bm.bimask_workspace_bytes(1, I, J, P)
    bm.bimask_perm_search(b["maskbits_f"], I, J, N, M, P, seed, None, b["perm"], b["best_idx"], b["counts"], b["ws"], ws_bytes)
    torch.cuda.synchronize()
    cands = O.candidates(seed, P, I)
    best, perm, cnt = O.perm_search(B, cands, N, M)
    assert np.array_equal(b["counts"].cpu().numpy(), cnt)
    assert int(b["best_idx"].item()) == best
    assert np.array_equal(b["perm"].cpu().numpy(), perm)
    # backward mask on the chosen permutation
    bm.bimask_bwd_mask(Wd, b["maskbits_f"], b["perm"], I, J, N, M, b["maskbits_b"], b["vals_b"], opt(b["meta_b"]),
                       opt(b["hw_meta_b"]))
    torch.cuda.synchronize()
    Bbar = O.backward_mask(W, B, perm, N, M)
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(Bbar))
    if pack:
        _, vals, meta = O.backward_operand(W, Bbar, perm)
        assert np.array_equal(u32(b["meta_b"]), meta)
        assert np.array_equal(u16(b["vals_b"]), vals)
    else:
        assert np.array_equal(u16(b["vals_b"]), O.dense_backward_operand(W, Bbar, perm))


@pytest.mark.parametrize("N,M", [(2, 8), (1, 8), (1, 16)])
def test_other_patterns_layer_step(N, M):
    I, J, T = 384, 512, 300
    W = inputs.make_weight(I, J, 100 + N + M)
    X = inputs.make_activation(T, J, 101)
    dY = inputs.make_activation(T, I, 102)
    b = run_layer_step(W, X, dY, N, M, 5, 17, do_search=True)
    ref = O.layer_step(W, X, dY, N, M, 5, 17, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy(), ref["Y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL


@pytest.mark.parametrize("N,M,I,J,T", [(4, 8, 384, 512, 300), (4, 8, 128, 1056, 100), (3, 8, 1024, 384, 1000),
                                       (4, 16, 96, 160, 129), (8, 8, 256, 256, 64)])
def test_unpackable_patterns_run_the_layer_step_on_dense_operands(N, M, I, J, T):
    """4:8 (and any pattern with more than two survivors in a group of four) has no sparse tensor-core
    format: the step runs the same masks and search and feeds dense masked operands to the products."""
    W = inputs.make_weight(I, J, 200 + N + M)
    X = inputs.make_activation(T, J, 201)
    dY = inputs.make_activation(T, I, 202)
    b = bm.alloc_layer_buffers(T, I, J, 5, dense=True)
    b["W"], b["X"], b["dY"] = dev(W), bits_dev(X), bits_dev(dY)
    b["meta_f"] = b["hw_meta_f"] = b["meta_b"] = b["hw_meta_b"] = None
    bm.bimask_layer_step(bm.make_layer_args(T, I, J, N, M, 5, 17, True, b))
    torch.cuda.synchronize()
    ref = O.layer_step(W, X, dY, N, M, 5, 17, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(ref["B"]))
    assert np.array_equal(u16(b["vals_f"]), O.dense_operand(W, ref["B"]))
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(ref["Bbar_p"]))
    assert np.array_equal(u16(b["vals_b"]), O.dense_backward_operand(W, ref["Bbar_p"], ref["perm"]))
    assert rel_err(b["Y"].float().cpu().numpy(), ref["Y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dX"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL
    # the stand-alone products accept the dense operand when no metadata image is given
    Y2 = torch.empty_like(b["Y"])
    bm.bimask_spmm_fwd(b["X"], b["vals_f"], None, T, I, J, Y2, b["status_word"])
    dX2 = torch.empty_like(b["dX"])
    bm.bimask_spmm_dgrad(b["dY"], b["perm"], b["vals_b"], None, T, I, J, dX2, b["ws"], b["ws"].numel(), b["status_word"])
    torch.cuda.synchronize()
    assert torch.equal(Y2, b["Y"]) and torch.equal(dX2, b["dX"])


def test_bounded_wait_reports_timeout_and_context_survives():
    """A wait on a barrier that nothing completes gives up after its budget (about a millisecond),
    reports through the status word and leaves the context usable."""
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    bm.bimask_debug_wait_probe(st)
    torch.cuda.synchronize()
    assert int(st.item()) == bm.binding.BIMASK_ETIMEOUT
    W = inputs.make_weight(64, 64, 1)
    _, b = run_fwd_mask(W, 2)                       # the device still works
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(O.forward_mask(W, 2, 4)))


@pytest.mark.parametrize("I,J,T", [(2176, 4128, 1040), (2048, 4096, 1024), (4224, 2080, 1265)])
def test_large_operand_sparse_kernel_ragged_shapes(I, J, T):
    """Operands of >= 2048 rows with >= 1024 tokens and k >= 4096 run on the kernel that pairs two row tiles per
    token tile: rows that do not fill the last 512-row tile, a ragged token tail and a k tail, forward and input gradient."""
    N, M = 2, 4
    W = inputs.make_weight(I, J, 900 + I % 97)
    X = inputs.make_activation(T, J, 901)
    dY = inputs.make_activation(T, I, 902)
    rng = np.random.default_rng(I + J)
    perm = rng.permutation(I).astype(np.int32)
    b = run_layer_step(W, X, dY, N, M, 2, 5, do_search=False, perm=perm)
    assert int(b["status_word"].item()) == 0
    B = O.forward_mask(W, N, M)
    Bbar = O.backward_mask(W, B, perm, N, M)
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(Bbar))
    assert rel_err(b["Y"].float().cpu().numpy(), O.spmm_fwd(X, W, B)) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), O.spmm_dgrad(dY, W, O.unpermute_rows(Bbar, perm))) <= TOL


def test_async_host_calls_with_alternating_buffer_sets():
    """Three device buffer sets used in turn, ten calls in flight before one wait, every call with its own
    inputs and its own host outputs: uploads, kernels and downloads of different calls overlap, and a set
    that comes round again must wait for the call that used it last.  Every result equals the blocking one."""
    shapes = [(1024, 1536, 900), (1536, 1024, 700), (2048, 512, 1100)]
    N, P = 2, 4
    sets, refs, outs = [], [], []
    for k, (I, J, T) in enumerate(shapes):
        b = bm.alloc_layer_buffers(T, I, J, P)
        b["W"] = torch.empty(I, J, device="cuda")
        b["X"] = torch.empty(T, J, dtype=torch.bfloat16, device="cuda")
        b["dY"] = torch.empty(T, I, dtype=torch.bfloat16, device="cuda")
        sets.append(b)
    calls = []
    for c in range(10):
        k = c % 3
        I, J, T = shapes[k]
        W = inputs.make_weight(I, J, 700 + c)
        X = inputs.make_activation(T, J, 800 + c)
        dY = inputs.make_activation(T, I, 900 + c)
        host = {"W": torch.from_numpy(W).pin_memory(),
                "X": torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).pin_memory(),
                "dY": torch.from_numpy(dY.view(np.int16)).view(torch.bfloat16).pin_memory(),
                "Y": torch.zeros(T, I, dtype=torch.bfloat16).pin_memory(),
                "dX": torch.zeros(T, J, dtype=torch.bfloat16).pin_memory(),
                "dW": torch.zeros(I, J, dtype=torch.float32).pin_memory(),
                "perm": torch.zeros(I, dtype=torch.int32).pin_memory(),
                "counts": torch.zeros(P, dtype=torch.int64).pin_memory()}
        calls.append((k, W, X, dY, host, torch.full((1,), -9, dtype=torch.int32).pin_memory()))
    for c, (k, W, X, dY, host, hst) in enumerate(calls):
        I, J, T = shapes[k]
        bm.bimask_layer_step_host_async(bm.make_layer_args(T, I, J, N, 4, P, 50 + c, True, sets[k]),
                                        bm.make_layer_args(T, I, J, N, 4, P, 50 + c, True, host), hst)
    bm.bimask_host_sync()
    for c, (k, W, X, dY, host, hst) in enumerate(calls):
        ref = run_layer_step(W, X, dY, N, 4, P, 50 + c, do_search=True)
        assert int(hst.item()) == 0, c
        assert torch.equal(host["perm"], ref["perm"].cpu()), c
        assert torch.equal(host["counts"], ref["counts"].cpu()), c
        assert torch.equal(host["Y"], ref["Y"].cpu()), c
        assert torch.equal(host["dX"], ref["dX"].cpu()), c
        assert torch.equal(host["dW"], ref["dW"].cpu()), c


def test_two_host_threads_on_their_own_streams():
    """Two host threads call the layer step at the same time, each on its own stream and buffers (the library's side
    streams, events and tensor-map cache are per host thread, its shared-memory attribute table per device and
    atomic): twelve steps each on alternating inputs, sizes on both sides of the side-stream threshold; every result
    equals that of the same step run alone."""
    import threading
    jobs = [(256, 384, 6000, 2), (1152, 384, 1500, 2), (64, 576, 300, 1), (512, 1184, 1568, 2)]
    refs, work = [], []
    for t, (I, J, T, N) in enumerate(jobs):
        ins = [(inputs.make_weight(I, J, 31 * t + v), inputs.make_activation(T, J, 37 * t + v),
                inputs.make_activation(T, I, 41 * t + v)) for v in range(2)]
        refs.append([run_layer_step(W, X, dY, N, 4, 4, 9 + t, do_search=True) for (W, X, dY) in ins])
        work.append(ins)
    torch.cuda.synchronize()
    results, errors = {}, []

    def worker(tid):
        try:
            st = torch.cuda.Stream()
            for t in (tid, tid + 2):                       # two jobs per thread, one after the other
                I, J, T, N = jobs[t]
                b = bm.alloc_layer_buffers(T, I, J, 4)
                dev_in = [(dev(W), bits_dev(X), bits_dev(dY)) for (W, X, dY) in work[t]]
                torch.cuda.synchronize()
                got = []
                for step in range(12):
                    b["W"], b["X"], b["dY"] = dev_in[step & 1]
                    bm.bimask_layer_step(bm.make_layer_args(T, I, J, N, 4, 4, 9 + t, True, b, stream=st))
                    if step >= 10:                         # keep the last two (one per input set)
                        st.synchronize()
                        got.append({k: b[k].clone() for k in ("perm", "counts", "Y", "dX", "dW", "maskbits_b", "status_word")})
                st.synchronize()
                results[t] = got
        except Exception as e:                             # surfaced by the main thread
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    for t in range(4):
        for v, got in enumerate(results[t]):
            ref = refs[t][v]
            assert int(got["status_word"].item()) == 0
            for k in ("perm", "counts", "maskbits_b", "Y", "dX", "dW"):
                assert torch.equal(got[k], ref[k]), (t, v, k)


@pytest.mark.parametrize("I,J,T", [(256, 384, 512), (64, 576, 3000), (256, 384, 6000), (64, 576, 16000), (1152, 384, 1500)])
def test_back_to_back_steps_on_reused_buffers(I, J, T):
    """Every kernel is launched as a programmatic dependent of the one before it and may begin before that one
    has finished; layers of more than a gigaflop (the last three shapes) also run parts of the step on side streams
    that fork from and join the caller's stream.  Steps on alternating inputs, enqueued back to back into the same
    buffers with no synchronisation in between, must give each step's own results: a kernel that read or wrote ahead
    of its dependency would pick up the other input's data."""
    N, M, P = 2, 4, 6
    sets = []
    for k in range(2):
        W = inputs.make_weight(I, J, 500 + k)
        X = inputs.make_activation(T, J, 510 + k)
        dY = inputs.make_activation(T, I, 520 + k)
        sets.append((W, X, dY, dev(W), bits_dev(X), bits_dev(dY), O.layer_step(W, X, dY, N, M, P, 40 + k)))
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"], b["X"], b["dY"] = torch.empty_like(sets[0][3]), torch.empty_like(sets[0][4]), torch.empty_like(sets[0][5])
    keep = {}
    for it in range(24):
        k = it & 1
        b["W"].copy_(sets[k][3]); b["X"].copy_(sets[k][4]); b["dY"].copy_(sets[k][5])
        bm.bimask_layer_step(bm.make_layer_args(T, I, J, N, M, P, 40 + k, True, b))
        if it >= 22:                                      # device-side copies of the last two steps' results
            keep[k] = {n: b[n].clone() for n in ("maskbits_f", "meta_f", "counts", "perm", "maskbits_b", "meta_b", "Y", "dX", "dW")}
    torch.cuda.synchronize()
    assert int(b["status_word"].item()) == 0
    for k in range(2):
        ref, got = sets[k][6], keep[k]
        assert np.array_equal(u32(got["maskbits_f"]), ref["maskbits_f"])
        assert np.array_equal(u32(got["meta_f"]), ref["meta_f"])
        assert np.array_equal(got["counts"].cpu().numpy(), ref["counts"])
        assert np.array_equal(got["perm"].cpu().numpy(), ref["perm"])
        assert np.array_equal(u32(got["maskbits_b"]), ref["maskbits_b"])
        assert np.array_equal(u32(got["meta_b"]), ref["meta_b"])
        for n in ("Y", "dX", "dW"):
            assert rel_err(got[n].float().cpu().numpy(), ref[n]) <= TOL, (k, n)


def _random_shapes(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n):
        I = 32 * int(rng.integers(1, 41))                 # 32 .. 1280
        J = 32 * int(rng.integers(1, 41))
        T = int(rng.integers(1, 2600))
        NM = [(2, 4), (1, 4), (2, 8), (1, 16), (4, 8)][int(rng.integers(0, 5))]
        out.append((I, J, T) + NM)
    return out


@pytest.mark.parametrize("I,J,T,N,M", _random_shapes(16, 20240607))
def test_layer_step_parity_on_drawn_shapes(I, J, T, N, M):
    """Shapes drawn at random (seeded): every kernel choice the dispatchers make below the large-operand kernels,
    ragged tiles in all three dimensions, packed and dense operands."""
    if J % M or I % M:
        J, I = J + (-J) % 64, I + (-I) % 64
    W = inputs.make_weight(I, J, I + 3 * J)
    X = inputs.make_activation(T, J, T + I)
    dY = inputs.make_activation(T, I, T + J)
    P, seed = 5, 77 + T
    b = run_layer_step(W, X, dY, N, M, P, seed, do_search=True) if N <= 2 else None
    if b is None:                                         # dense masked operands (no 2:4 form)
        b = bm.alloc_layer_buffers(T, I, J, P, dense=True)
        b["W"], b["X"], b["dY"] = dev(W), bits_dev(X), bits_dev(dY)
        b["meta_f"] = b["hw_meta_f"] = b["meta_b"] = b["hw_meta_b"] = None
        bm.bimask_layer_step(bm.make_layer_args(T, I, J, N, M, P, seed, True, b))
        torch.cuda.synchronize()
    ref = O.layer_step(W, X, dY, N, M, P, seed, do_search=True)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), O.pack_bits(ref["B"]))
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), O.pack_bits(ref["Bbar_p"]))
    for n in ("Y", "dX", "dW"):
        assert rel_err(b[n].float().cpu().numpy(), ref[n]) <= TOL, n


@pytest.mark.parametrize("T", [700, 6000])
def test_layer_step_captured_in_a_cuda_graph(T):
    """The entry points enqueue kernels only (programmatic dependent launches included; at T = 6000 also the forks to
    and joins from the side streams of a layer above a gigaflop), so a step can be captured once and replayed: the
    replay on new contents of the same buffers must give that input's results."""
    I, J, N, M, P = 256, 384, 2, 4, 6
    sets = [(inputs.make_weight(I, J, 600 + k), inputs.make_activation(T, J, 610 + k), inputs.make_activation(T, I, 620 + k))
            for k in range(2)]
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"], b["X"], b["dY"] = dev(sets[0][0]), bits_dev(sets[0][1]), bits_dev(sets[0][2])
    args = bm.make_layer_args(T, I, J, N, M, P, 9, True, b)
    bm.bimask_layer_step(args)                            # first call: kernel attributes and tensor maps
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        args.stream = torch.cuda.current_stream().cuda_stream
        bm.bimask_layer_step(args)
    for k in (1, 0, 1):
        b["W"].copy_(dev(sets[k][0])); b["X"].copy_(bits_dev(sets[k][1])); b["dY"].copy_(bits_dev(sets[k][2]))
        graph.replay()
    torch.cuda.synchronize()
    ref = O.layer_step(sets[1][0], sets[1][1], sets[1][2], N, M, P, 9)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    for n in ("Y", "dX", "dW"):
        assert rel_err(b[n].float().cpu().numpy(), ref[n]) <= TOL, n
