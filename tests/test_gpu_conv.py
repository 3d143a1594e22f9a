"""GPU parity for the 3x3 convolution layer step (bimask_conv_layer_step) against the oracle's
direct convolutions: integer results bit for bit, the three products within the GEMM tolerance.
Shapes cover images smaller and larger than a pixel patch, ragged patch edges, batch sizes that do
not fill a patch group, channel counts on both sides of the implicit form's limits."""
import numpy as np
import pytest
import torch

import paper_2302_06058_b200 as bm
from oracle import bimask_oracle as O
from paper_2302_06058_b200 import inputs
from tests.gpu_util import bits_dev, dev, rel_err, u16, u32

pytestmark = pytest.mark.gpu
TOL = 2e-2


def conv_case(NB, H, W, C, I, seed):
    Wt = inputs.make_weight(I, 9 * C, seed)
    x = inputs.make_activation(NB * H * W, C, seed + 1).reshape(NB, H, W, C)
    dy = inputs.make_activation(NB * H * W, I, seed + 2).reshape(NB, H, W, I)
    return Wt, x, dy


def run_conv_step(Wt, x, dy, N, M, P, seed, mode, do_search=True, stride=1):
    NB, H, W, C = x.shape
    I = Wt.shape[0]
    T, J = dy.shape[0] * dy.shape[1] * dy.shape[2], 9 * C
    b = bm.alloc_layer_buffers(T, I, J, P)
    b["W"], b["X"], b["dY"] = dev(Wt), bits_dev(x), bits_dev(dy)
    b["dX"] = torch.empty(NB, H, W, C, dtype=torch.bfloat16, device="cuda")
    b["ws"] = torch.empty(bm.bimask_conv_workspace_bytes(NB, H, W, C, I, P, stride), dtype=torch.uint8, device="cuda")
    largs = bm.make_layer_args(T, I, J, N, M, P, seed, do_search, b)
    bm.bimask_conv_layer_step(bm.make_conv_args(largs, NB, H, W, C, mode, stride))
    torch.cuda.synchronize()
    return b


SHAPES = [(2, 9, 11, 32, 64), (3, 14, 14, 64, 128), (5, 7, 7, 128, 128), (1, 20, 17, 128, 256), (2, 28, 28, 128, 384),
          (1, 33, 8, 256, 128), (2, 7, 7, 128, 128), (1, 14, 14, 256, 512), (3, 5, 4, 192, 320),
          # column matrices above 16 MiB: AUTO takes the implicit form where the channel counts allow it
          (20, 28, 28, 64, 128), (8, 28, 28, 192, 320), (6, 40, 36, 128, 256)]


@pytest.mark.parametrize("NB,H,W,C,I", SHAPES)
@pytest.mark.parametrize("mode", [bm.binding.CONV_EXPLICIT, bm.binding.CONV_AUTO])
def test_conv_layer_step_against_oracle(NB, H, W, C, I, mode):
    N, M, P, seed = 2, 4, 4, 21
    Wt, x, dy = conv_case(NB, H, W, C, I, 300 + NB + H + C)
    b = run_conv_step(Wt, x, dy, N, M, P, seed, mode)
    ref = O.conv_layer_step(Wt, x, dy, N, M, P, seed)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(u16(b["vals_f"]), ref["vals_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy().reshape(NB, H, W, I), ref["y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dx"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL


def test_conv_other_pattern_and_dense_fallback():
    NB, H, W, C, I = 2, 10, 12, 64, 128
    Wt, x, dy = conv_case(NB, H, W, C, I, 77)
    for (N, M) in [(1, 4), (2, 8)]:
        b = run_conv_step(Wt, x, dy, N, M, 3, 5, bm.binding.CONV_AUTO)
        ref = O.conv_layer_step(Wt, x, dy, N, M, 3, 5)
        assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
        assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
        assert rel_err(b["Y"].float().cpu().numpy().reshape(NB, H, W, I), ref["y"]) <= TOL
        assert rel_err(b["dX"].float().cpu().numpy(), ref["dx"]) <= TOL
        assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL


@pytest.mark.parametrize("N,M", [(1, 4), (2, 8), (1, 16)])
def test_conv_implicit_form_other_patterns(N, M):
    NB, H, W, C, I = 2, 10, 12, 128, 128
    Wt, x, dy = conv_case(NB, H, W, C, I, 78)
    b = run_conv_step(Wt, x, dy, N, M, 3, 5, bm.binding.CONV_IMPLICIT)
    ref = O.conv_layer_step(Wt, x, dy, N, M, 3, 5)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy().reshape(NB, H, W, I), ref["y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dx"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL


@pytest.mark.parametrize("NB,H,W,C,I", [(2, 9, 11, 32, 64), (3, 14, 14, 64, 128), (2, 56, 56, 128, 128), (4, 28, 27, 256, 256),
                                        (1, 8, 8, 64, 64), (5, 15, 9, 192, 96), (32, 56, 56, 64, 64), (2, 7, 7, 128, 128), (3, 1, 5, 128, 64),
                                        (2, 14, 13, 512, 256)])
def test_conv_stride_2(NB, H, W, C, I):
    """ResNet's down-sampling 3x3 convolutions (stride 2): odd and even image sizes, images smaller than a pixel box,
    a batch that makes the automatic mode go implicit.  The forward product and the weight gradient have an implicit
    form (tensor loads that take every second pixel); the input gradient runs as four stride-1 products, one per parity
    class of the input pixels (C = 64 or a multiple of 128; explicit otherwise)."""
    N, M, P, seed = 2, 4, 4, 23
    Ho, Wo = O.conv_out_size(H, 2), O.conv_out_size(W, 2)
    Wt = inputs.make_weight(I, 9 * C, 330 + H)
    x = inputs.make_activation(NB * H * W, C, 331).reshape(NB, H, W, C)
    dy = inputs.make_activation(NB * Ho * Wo, I, 332).reshape(NB, Ho, Wo, I)
    ref = O.conv_layer_step(Wt, x, dy, N, M, P, seed, stride=2)
    modes = [bm.binding.CONV_EXPLICIT, bm.binding.CONV_AUTO] + ([bm.binding.CONV_IMPLICIT] if C % 64 == 0 else [])
    launches = {}
    for mode in modes:
        n0 = bm.bimask_launch_count()
        b = run_conv_step(Wt, x, dy, N, M, P, seed, mode, stride=2)
        launches[mode] = bm.bimask_launch_count() - n0
        assert int(b["status_word"].item()) == 0
        assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
        assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
        assert rel_err(b["Y"].float().cpu().numpy().reshape(NB, Ho, Wo, I), ref["y"]) <= TOL, mode
        assert rel_err(b["dX"].float().cpu().numpy(), ref["dx"]) <= TOL, mode
        assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL, mode
    if C % 64 == 0:      # no unfold pass in the implicit form; four input-gradient launches instead of product + fold
        assert launches[bm.binding.CONV_IMPLICIT] <= launches[bm.binding.CONV_EXPLICIT] + 2
    else:
        with pytest.raises(bm.BimaskError) as e:
            run_conv_step(Wt, x, dy, N, M, P, seed, bm.binding.CONV_IMPLICIT, stride=2)
        assert e.value.code == -2


def test_conv_bad_arguments_launch_nothing():
    NB, H, W, C, I = 1, 8, 8, 32, 32
    Wt, x, dy = conv_case(NB, H, W, C, I, 1)
    T, J = NB * H * W, 9 * C
    b = bm.alloc_layer_buffers(T, I, J, 2)
    b["W"], b["X"], b["dY"] = dev(Wt), bits_dev(x), bits_dev(dy)
    b["dX"] = torch.empty(NB, H, W, C, dtype=torch.bfloat16, device="cuda")
    n0 = bm.bimask_launch_count()
    largs = bm.make_layer_args(T, I, J, 2, 4, 2, 1, True, b)          # workspace sized for the linear layer: too small
    with pytest.raises(bm.BimaskError) as e:
        bm.bimask_conv_layer_step(bm.make_conv_args(largs, NB, H, W, C, 0))
    assert e.value.code == -1 and "workspace" in str(e.value)
    b["ws"] = torch.empty(bm.bimask_conv_workspace_bytes(NB, H, W, C, I, 2), dtype=torch.uint8, device="cuda")
    largs = bm.make_layer_args(T, I, J, 2, 4, 2, 1, True, b)
    for kw in (dict(H=7), dict(C=48), dict(mode=5), dict(stride=2)):
        geo = dict(NB=NB, H=H, W=W, C=C, mode=0, stride=1)
        geo.update(kw)
        with pytest.raises(bm.BimaskError) as e:
            bm.bimask_conv_layer_step(bm.make_conv_args(largs, geo["NB"], geo["H"], geo["W"], geo["C"], geo["mode"], geo["stride"]))
        assert e.value.code == -1
    with pytest.raises(bm.BimaskError) as e:                             # C = 32 cannot take the implicit form
        bm.bimask_conv_layer_step(bm.make_conv_args(largs, NB, H, W, C, bm.binding.CONV_IMPLICIT))
    assert e.value.code == -2
    assert bm.bimask_launch_count() == n0


@pytest.mark.parametrize("NB,H,W,C,I", [(5, 7, 7, 128, 128), (1, 20, 17, 128, 256), (2, 28, 28, 128, 384),
                                        (1, 33, 8, 256, 128), (1, 14, 14, 256, 512), (4, 56, 56, 128, 128),
                                        # 64 input channels (taps start in the middle of a metadata block) and output
                                        # channel counts that are not multiples of 128 (ragged k tiles per tap)
                                        (4, 56, 56, 64, 64), (2, 20, 20, 64, 96), (2, 14, 14, 128, 192),
                                        (1, 16, 16, 256, 160), (3, 9, 9, 64, 320)])
def test_conv_implicit_form_builds_no_column_matrix(NB, H, W, C, I):
    N, M, P, seed = 2, 4, 4, 33
    Wt, x, dy = conv_case(NB, H, W, C, I, 500 + H + C)
    n0 = bm.bimask_launch_count()
    b = run_conv_step(Wt, x, dy, N, M, P, seed, bm.binding.CONV_IMPLICIT)
    n_imp = bm.bimask_launch_count() - n0
    b2 = run_conv_step(Wt, x, dy, N, M, P, seed, bm.binding.CONV_EXPLICIT)
    n_exp = bm.bimask_launch_count() - n0 - n_imp
    assert n_exp - n_imp >= 1                      # the unfold and fold passes are gone (the split-K plans may differ by one launch)
    ref = O.conv_layer_step(Wt, x, dy, N, M, P, seed)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    for got in (b, b2):
        assert rel_err(got["Y"].float().cpu().numpy().reshape(NB, H, W, I), ref["y"]) <= TOL
        assert rel_err(got["dX"].float().cpu().numpy(), ref["dx"]) <= TOL
        assert rel_err(got["dW"].cpu().numpy(), ref["dW"]) <= TOL


@pytest.mark.parametrize("H,W,C,I", [(56, 56, 64, 64), (28, 28, 128, 128), (14, 14, 256, 256), (7, 7, 512, 512)])
def test_conv_resnet50_layers_at_batch_32(H, W, C, I):
    """ResNet-50's four 3x3 layer shapes at the batch size bench.py --conv times, automatic form (implicit for the
    first three, whose column matrices exceed 16 MiB; explicit for 7 x 7)."""
    NB, N, M, P, seed = 32, 2, 4, 32, 45
    Wt, x, dy = conv_case(NB, H, W, C, I, 640 + H)
    b = run_conv_step(Wt, x, dy, N, M, P, seed, bm.binding.CONV_AUTO)
    ref = O.conv_layer_step(Wt, x, dy, N, M, P, seed)
    assert int(b["status_word"].item()) == 0
    assert np.array_equal(u32(b["maskbits_f"]), ref["maskbits_f"])
    assert np.array_equal(b["counts"].cpu().numpy(), ref["counts"])
    assert np.array_equal(b["perm"].cpu().numpy(), ref["perm"])
    assert np.array_equal(u32(b["maskbits_b"]), ref["maskbits_b"])
    assert np.array_equal(u16(b["vals_b"]), ref["vals_b"])
    assert rel_err(b["Y"].float().cpu().numpy().reshape(NB, H, W, I), ref["y"]) <= TOL
    assert rel_err(b["dX"].float().cpu().numpy(), ref["dx"]) <= TOL
    assert rel_err(b["dW"].cpu().numpy(), ref["dW"]) <= TOL
