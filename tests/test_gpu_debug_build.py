"""The bounds-reporting build (libbimask_debug.so, -DBIMASK_DEBUG) on the GPU.

Every kernel that turns a caller-supplied row index into an address clamps it (both builds), so a bad permutation
can never fault; the debug build also records the first offender for bimask_debug_status().  The checks run in a
child process because the binding holds one library per process.  compute-sanitizer is not available on this machine:
this build, the ragged / small shapes below and the element-wise comparison with the CPU oracle stand in for it."""
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_CHILD = r"""
import sys
import numpy as np, torch
sys.path.insert(0, %r)
sys.path.insert(0, %r)
import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from gpu_util import dev, run_fwd_mask, run_layer_step, u32, u16, rel_err

assert bm.binding.LIB_PATH.endswith("libbimask_debug.so")
rng = np.random.default_rng(3)

# 1. ragged and small layer steps: bit-exact integers, products within tolerance, and a clean record
for (I, J, T, N, P) in [(32, 32, 1, 2, 3), (96, 160, 127, 1, 5), (256, 256, 129, 2, 8), (512, 1184, 200, 2, 4),
                        (1152, 384, 333, 2, 6)]:
    W = rng.standard_normal((I, J)).astype(np.float32)
    X = O.bf16_bits(rng.standard_normal((T, J)).astype(np.float32))
    dY = O.bf16_bits(rng.standard_normal((T, I)).astype(np.float32))
    b = run_layer_step(W, X, dY, N, 4, P, 77)
    ref = O.layer_step(W, X, dY, N, 4, P, 77)
    assert int(b["status_word"].item()) == 0
    for k in ("maskbits_f", "meta_f", "maskbits_b", "meta_b"):
        assert np.array_equal(u32(b[k]), ref[k]), (k, I, J)
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"]) and np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    for k in ("Y", "dX", "dW"):
        assert rel_err(b[k].float().cpu().numpy(), ref[k]) <= 2e-2, (k, I, J)
    assert bm.bimask_debug_status() == [0, 0, 0, 0], (I, J)

# 2. a permutation with one entry out of range: nothing faults, the result is that of the clamped entry, and the
#    record names the site (1 = backward mask), the index and the bound
I, J = 256, 256
W = rng.standard_normal((I, J)).astype(np.float32)
Wd, b = run_fwd_mask(W, 2)
perm = rng.permutation(I).astype(np.int32)
bad = perm.copy(); bad[5] = I + 3
bm.bimask_bwd_mask(Wd, b["maskbits_f"], dev(bad), I, J, 2, 4, b["maskbits_b"], b["vals_b"], b["meta_b"], b["hw_meta_b"])
rec = bm.bimask_debug_status()
assert rec == [bm.binding.BIMASK_EBOUNDS, 1, I + 3, I], rec
clamped = bad.copy(); clamped[5] = I - 1
B = O.forward_mask(W, 2, 4)
bits, vals, meta = O.backward_operand(W, O.backward_mask(W, B, clamped, 2, 4), clamped)
assert np.array_equal(u32(b["maskbits_b"]), bits) and np.array_equal(u16(b["vals_b"]), vals)
assert bm.bimask_debug_status() == [0, 0, 0, 0]          # reading the record cleared it

# 3. a candidate with a negative entry: site 2 (count kernel)
cands = np.stack([rng.permutation(I) for _ in range(3)]).astype(np.int32)
cands[1, 9] = -4
ws = torch.empty(bm.bimask_workspace_bytes(1, I, J, 3), dtype=torch.uint8, device="cuda")
bp = torch.empty(I, dtype=torch.int32, device="cuda"); bi = torch.empty(1, dtype=torch.int32, device="cuda")
cnt = torch.empty(3, dtype=torch.int64, device="cuda")
bm.bimask_perm_search(b["maskbits_f"], I, J, 2, 4, 3, 0, dev(cands), bp, bi, cnt, ws, ws.numel())
rec = bm.bimask_debug_status()
assert rec == [bm.binding.BIMASK_EBOUNDS, 2, -4, I], rec
print("debug build ok")
"""


@pytest.mark.gpu
def test_ragged_shapes_and_bad_indices_under_the_debug_build():
    env = dict(os.environ, BIMASK_LIBRARY="debug")
    out = subprocess.run([sys.executable, "-c", _CHILD % (ROOT, os.path.join(ROOT, "tests"))], cwd=ROOT, env=env,
                         text=True, capture_output=True, timeout=900)
    assert out.returncode == 0 and "debug build ok" in out.stdout, out.stdout[-2000:] + out.stderr[-4000:]


def test_release_build_has_no_record():
    import paper_2302_06058_b200 as bm
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_debug_status()
    assert e.value.code == bm.binding.BIMASK_EUNSUPPORTED
