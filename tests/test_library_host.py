"""CPU-only checks of the boundary: the shared library loads, exports every symbol the header
declares, and the host-side logic that needs no GPU (size queries, argument validation, the
multi-process replica arithmetic of the benchmark) behaves."""
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def bm():
    from paper_2302_06058_b200 import build
    build.build()
    import paper_2302_06058_b200 as m
    m.lib()
    return m


def header_symbols():
    text = open(os.path.join(ROOT, "include", "bimask.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bimask_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(bm):
    names = header_symbols()
    assert "bimask_layer_step" in names and "bimask_spmm_dgrad" in names and len(names) >= 12
    L = bm.lib()
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(bm.binding.EXPORTS)


def test_binding_has_same_names(bm):
    for n in header_symbols():
        assert callable(getattr(bm, n)), n


def test_size_queries(bm):
    assert bm.bimask_hw_meta_bytes(128, 128) == 2048
    assert bm.bimask_hw_meta_bytes(64, 576) == 5 * 2048            # rows and k are padded to 128
    assert bm.bimask_hw_meta_bytes(16384, 4096) == 16384 * 4096 // 8
    assert bm.bimask_hw_meta_bytes(0, 128) == 0
    ws = bm.bimask_workspace_bytes(8192, 16384, 4096, 128)
    assert ws >= 128 * 16384 * 4 + 8192 * 16384 * 2                # candidates + permuted dY
    small = bm.bimask_workspace_bytes(100352, 64, 576, 32)         # few tiles => split-K partials
    assert small >= 32 * 64 * 4 + 100352 * 64 * 2 + 2 * 64 * 576 * 4
    assert bm.bimask_workspace_bytes(8, 0, 64, 1) == 0


def test_validation_happens_before_any_cuda_call(bm):
    """Bad arguments are rejected on the host: these calls work (and fail cleanly) without a GPU."""
    L = bm.lib()
    rc = L.bimask_fwd_mask(None, 64, 64, 2, 4, None, None, None, None, None)
    assert rc == bm.binding.BIMASK_EINVAL and "null" in bm.bimask_last_error()
    assert L.bimask_fwd_mask(16, 64, 60, 2, 4, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_fwd_mask(16, 64, 64, 2, 32, 16, 16, 16, 16, None) == bm.binding.BIMASK_EUNSUPPORTED     # M = 32
    assert L.bimask_fwd_mask(16, 64, 64, 4, 8, 16, 16, 16, 16, None) == bm.binding.BIMASK_EUNSUPPORTED      # 4:8 cannot be packed
    assert "dense masked operand" in bm.bimask_last_error()
    assert L.bimask_fwd_mask(16, 64, 64, 3, 4, 16, 16, 16, 16, None) == bm.binding.BIMASK_EUNSUPPORTED
    assert L.bimask_fwd_mask(16, 64, 64, 0, 4, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_fwd_mask(20, 64, 64, 2, 4, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL   # misaligned
    assert L.bimask_perm_search(16, 64, 64, 2, 4, 0, 1, None, 16, 16, 16, 16, 1 << 20, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_perm_search(16, 1 << 24, 64, 2, 4, 2, 1, None, 16, 16, 16, 16, 1 << 30, None) == bm.binding.BIMASK_EUNSUPPORTED
    assert L.bimask_perm_search(16, 64, 64, 2, 4, 2, 1, None, 16, 16, 16, 16, 8, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_spmm_fwd(16, 16, 16, 0, 64, 64, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_wgrad(16, 16, 8, 64, 64, None, None, 0, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_layer_step(None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_train_step(None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_conv_layer_step(None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_perm_refine(16, 64, 64, 2, 4, 2, 1, 16, None, None, 1 << 20, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_perm_refine(16, 64, 64, 2, 4, 2, 1, 16, None, 16, 8, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_perm_refine(16, 64, 64, 5, 8, 2, 1, 16, None, 16, 1 << 20, None) == bm.binding.BIMASK_EUNSUPPORTED
    assert bm.bimask_refine_workspace_bytes(16384, 4, 32) >= 32 * 16384 * 4 + 8192 * 4 + 4096 * 8
    assert bm.bimask_conv_workspace_bytes(32, 56, 56, 64, 64, 100) > 2 * 32 * 56 * 56 * 576 * 2
    assert bm.bimask_conv_workspace_bytes(0, 56, 56, 64, 64, 100) == 0
    assert L.bimask_bwd_mask_criterion(16, None, 16, 16, 64, 64, 2, 4, 7, 0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_bwd_mask_criterion(16, None, 16, 16, 64, 64, 2, 4, 1, 0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert "needs S" in bm.bimask_last_error()
    assert L.bimask_bwd_mask_criterion(16, None, 16, 16, 64, 64, 4, 8, 3, 0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EUNSUPPORTED
    assert L.bimask_sgd_fwd_mask(16, None, None, 64, 64, 2, 4, 0.1, 0.9, 0.0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_sgd_fwd_mask(16, 16, 20, 64, 64, 2, 4, 0.1, 0.9, 0.0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_sgd_fwd_mask(16, 16, 16, 64, 64, 2, 4, float("nan"), 0.9, 0.0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EINVAL
    assert L.bimask_sgd_fwd_mask(16, 16, 16, 64, 64, 4, 8, 0.1, 0.9, 0.0, 16, 16, 16, 16, None) == bm.binding.BIMASK_EUNSUPPORTED
    with pytest.raises(bm.BimaskError):
        bm.bimask_fwd_mask(None, 64, 64, 2, 4, None, None, None, None, stream=0)


def test_product_path_does_not_import_the_oracle():
    code = ("import sys; import paper_2302_06058_b200 as bm; bm.lib(); "
            "assert not any(m.startswith('oracle') for m in sys.modules), 'oracle imported'")
    subprocess.check_call([sys.executable, "-c", code], cwd=ROOT)
    for root, _, files in os.walk(os.path.join(ROOT, "paper_2302_06058_b200")):
        for f in files:
            if f.endswith(".py"):
                text = open(os.path.join(root, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle", text, flags=re.M), f


def test_missing_library_fails_loudly(tmp_path):
    code = ("import paper_2302_06058_b200.binding as b; b.LIB_PATH = r'%s'; b._lib = None\n"
            "try:\n    b.lib()\nexcept RuntimeError as e:\n    assert 'missing' in str(e); print('raised')\n"
            % str(tmp_path / "nope.so"))
    out = subprocess.check_output([sys.executable, "-c", code], cwd=ROOT, text=True)
    assert "raised" in out


_WORKER = r"""
import os, sys, json
import torch.distributed as dist
sys.path.insert(0, %r)
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# every rank times its own replica; bench.py's own helpers reduce the timings (max over ranks) and form the value
dist.barrier()
ms, other = bench.max_over_ranks([10.0 + 5.0 * rank, 7.0 - rank], world)
value = bench.job_value(world, 2, 4, ms)
if rank == 0:
    print(json.dumps({"ms": ms, "other": other, "value": value}))
dist.destroy_process_group()
"""


def test_replica_aggregation_world_size_2(tmp_path):
    """The multi-GPU path is N independent replicas: no collective touches the data; only the timings are reduced
    (max over ranks) and the value is world * layers * steps / that time.  Runs the functions bench.py uses."""
    script = tmp_path / "worker.py"
    script.write_text(_WORKER % ROOT)
    out = subprocess.check_output(
        [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
         "--master-addr", "127.0.0.1", "--master-port", "29731", str(script)],
        cwd=ROOT, text=True, stderr=subprocess.STDOUT, timeout=300)
    line = [l for l in out.splitlines() if l.startswith("{")][-1]
    import json
    d = json.loads(line)
    assert d["ms"] == 15.0 and d["other"] == 7.0
    assert abs(d["value"] - 2 * 2 * 4 / 0.015) < 1e-6


def test_clock_regime_picks_the_peak():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.clock_regime({"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, 0.08) == "burst"
    assert bench.clock_regime({"sm_mhz": 1965.0, "sm_max_mhz": 1965.0}, 6.0) == "sustained"
    assert bench.clock_regime({"sm_mhz": 1380.0, "sm_max_mhz": 1965.0}, 0.08) == "sustained"
    assert bench.clock_regime({"sm_mhz": None, "sm_max_mhz": None}) == "sustained"
    assert bench.job_value(2, 2, 4, 15.0) == 2 * 2 * 4 / 0.015


def test_bench_reference_arm_runs_on_cpu():
    out = subprocess.check_output([sys.executable, "bench.py", "--impl", "reference", "--config", "1", "--steps", "1",
                                   "--warmup", "0"], cwd=ROOT, text=True, timeout=600)
    import json
    d = json.loads(out.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["value"] > 0 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0
