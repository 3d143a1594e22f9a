"""bimask_perm_search_static: the workspace-free permutation search.

Some programs that embed this library cannot allocate device memory when they call it (their
runtime owns the whole GPU heap, or they are only lent pointers).  For them the search keeps its
generated candidates in an array built into the library.  This test calls that entry point through
the C ABI twice in a row -- the second time with a smaller problem, so that the shared array still
holds entries of the first call -- and requires exactly the results of bimask_perm_search (all
outputs are integers, so the comparison is bit for bit).  The reference here is the workspace entry
point, not the CPU oracle: that one is checked against the oracle in tests/test_gpu_parity.py
(generated candidates, counts, chosen permutation), so agreement with it carries the parity over."""
import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm

pytestmark = pytest.mark.gpu


def _random_maskbits(I, J, seed):
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    w = torch.randint(-2**31, 2**31 - 1, (I, J // 32), generator=g, dtype=torch.int64).to(torch.int32)
    return w.cuda()


def _both(I, J, N, P, seed):
    bits = _random_maskbits(I, J, 100 + I + P)
    out = []
    for which in ("workspace", "static"):
        best_perm = torch.full((I,), -1, dtype=torch.int32, device="cuda")
        best_idx = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        counts = torch.full((P,), -1, dtype=torch.int64, device="cuda")
        if which == "workspace":
            ws_bytes = bm.bimask_workspace_bytes(1, I, J, P)
            ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")
            bm.bimask_perm_search(bits, I, J, N, 4, P, seed, None, best_perm, best_idx, counts, ws, ws_bytes)
        else:
            bm.bimask_perm_search_static(bits, I, J, N, 4, P, seed, best_perm, best_idx, counts)
        torch.cuda.synchronize()
        out.append((best_perm.cpu().numpy(), int(best_idx.item()), counts.cpu().numpy()))
    return out


def test_static_search_matches_workspace_search_twice_in_a_row():
    for (I, J, N, P, seed) in [(2048, 512, 2, 24, 7), (512, 256, 1, 9, 8)]:
        (perm_a, idx_a, cnt_a), (perm_b, idx_b, cnt_b) = _both(I, J, N, P, seed)
        assert np.array_equal(cnt_a, cnt_b)
        assert idx_a == idx_b
        assert np.array_equal(perm_a, perm_b)
        assert np.array_equal(np.sort(perm_b), np.arange(I))


def test_static_search_rejects_sizes_beyond_its_array():
    limit = bm.bimask_perm_search_static_max_entries()
    assert limit == 2 * 1024 * 1024
    I, J = 16384, 64
    P = limit // I + 1
    bits = torch.zeros(I, J // 32, dtype=torch.int32, device="cuda")
    best_perm = torch.empty(I, dtype=torch.int32, device="cuda")
    best_idx = torch.empty(1, dtype=torch.int32, device="cuda")
    counts = torch.empty(P, dtype=torch.int64, device="cuda")
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_perm_search_static(bits, I, J, 2, 4, P, 1, best_perm, best_idx, counts)
    assert e.value.code == bm.binding.BIMASK_EUNSUPPORTED
    assert "exceed" in bm.bimask_last_error()
    # the largest size that fits is accepted
    P = limit // I
    counts = torch.empty(P, dtype=torch.int64, device="cuda")
    bm.bimask_perm_search_static(bits, I, J, 2, 4, P, 1, best_perm, best_idx, counts)
    torch.cuda.synchronize()
    assert int(counts.min().item()) == (I // 4) * J       # an all-zero mask: every block is eligible
