"""Kernel-by-kernel parity with the PLAIN float64 oracle, through the C ABI.

Every contraction / stencil kernel path of the library runs here as a stage of its own that has no
activation: with no ReLU/ReLU6 mask there is no binary decision that a rounding difference could flip, so
bfloat16 storage with float32 accumulation must meet the stated tolerance against the plain definition
directly: max|gpu-ref| / max|ref| <= 2e-2 (1e-4 in float32 storage) on the stage output, the input gradient,
every accumulated parameter gradient and every updated parameter, with no outlier allowance and no
diagnostic criterion.  Sizes cover partial tiles and, for the persistent kernels, more than one tile per CTA
(more than 148 x 128 pixels).  The kernel trace shows that the intended kernel is the one that ran."""
import numpy as np
import pytest

import stage_inputs as si
from harness import CONTRACT, MIRROR, bf16_store, compare, gpu_round, make_inputs, oracle_round, summary

pytestmark = pytest.mark.gpu

# name: (net, h, w, B, M, loss, kernels that must appear in the bfloat16 trace)
PW = ("pw_fwd_tcgen05", "pw_bwd_data_tcgen05", "pw_bwd_weight_tcgen05")
C3 = ("conv3x3_fwd_tcgen05", "conv3x3_bwd_data_tcgen05", "conv3x3_bwd_weight_tcgen05")
DW = ("dw_fwd",)
CASES = {
    # pointwise, K and N <= 256: the persistent pipelines; 2 x 101 x 97 = 19 594 pixels = 153.1 tiles of 128
    "pw_24_144": (si.single_unit_net("conv", 24, 144), 101, 97, 2, 2, "mse", PW),
    "pw_144_24": (si.single_unit_net("conv", 144, 24), 101, 97, 2, 2, "mse", PW),
    "pw_64_256": (si.single_unit_net("conv", 64, 256), 57, 43, 2, 1, "mse", PW),
    "pw_256_64": (si.single_unit_net("conv", 256, 64), 57, 43, 2, 1, "mse", PW),
    "pw_24_144_bn": (si.single_unit_net("conv", 24, 144, bn=True), 101, 97, 2, 2, "mse", PW),
    "pw_256_64_bn": (si.single_unit_net("conv", 256, 64, bn=True), 57, 43, 2, 1, "mse", PW),
    # pointwise with 512 channels on one side (ResNet conv3_x)
    "pw_128_512": (si.single_unit_net("conv", 128, 512), 29, 27, 3, 1, "mse", PW),
    "pw_512_128": (si.single_unit_net("conv", 512, 128), 29, 27, 3, 1, "mse", PW),
    "pw_512_128_bn": (si.single_unit_net("conv", 512, 128, bn=True), 29, 27, 3, 1, "mse", PW),
    "pw_320_1280_bn": (si.single_unit_net("conv", 320, 1280, bn=True), 7, 7, 5, 1, "mse", PW),
    # weight gradient on channel sub-ranges with the BatchNorm-backward transform on the wide side: four sub-ranges of 128
    # (512 channels), two of 192 (384 channels, where a quarter is no multiple of 64)
    "pw_128_512_bn": (si.single_unit_net("conv", 128, 512, bn=True), 29, 27, 3, 1, "mse", PW),
    "pw_128_384_bn": (si.single_unit_net("conv", 128, 384, bn=True), 23, 21, 3, 1, "mse", PW),
    # strided 1x1 (projection shortcut) on an odd-sized map
    "pw_s2_64_128": (si.single_unit_net("conv", 64, 128, stride=2), 13, 11, 3, 2, "mse", PW),
    "pw_s2_256_512_bn": (si.single_unit_net("conv", 256, 512, stride=2, bn=True), 13, 11, 3, 1, "mse", PW),
    # dense 3x3, stride 1
    "c3_64_64": (si.single_unit_net("conv", 64, 64, k=3), 23, 19, 3, 2, "mse", C3),
    "c3_64_64_bn": (si.single_unit_net("conv", 64, 64, k=3, bn=True), 23, 19, 3, 2, "mse", C3),
    "c3_64_64_56": (si.single_unit_net("conv", 64, 64, k=3), 56, 56, 8, 1, "mse", C3),
    "c3_128_128": (si.single_unit_net("conv", 128, 128, k=3), 28, 28, 3, 1, "mse", C3),
    "c3_128_128_bn": (si.single_unit_net("conv", 128, 128, k=3, bn=True), 15, 14, 3, 2, "mse", C3),
    "c3_64_128": (si.single_unit_net("conv", 64, 128, k=3), 15, 14, 3, 1, "mse", C3),
    # pipelined 3x3 kernels at their edges: a map narrower than one MMA row tile and shorter than a tile of image rows, a
    # last tile that runs past the bottom row, a single image, more tiles than CTAs (several windows per CTA)
    "c3_64_64_7x7_bn": (si.single_unit_net("conv", 64, 64, k=3, bn=True), 7, 7, 5, 1, "mse", C3),
    "c3_128_64_ragged_rows": (si.single_unit_net("conv", 128, 64, k=3, bn=True), 9, 61, 1, 2, "mse", C3),
    "c3_64_64_many_tiles_bn": (si.single_unit_net("conv", 64, 64, k=3, bn=True), 60, 33, 11, 1, "mse", C3),
    # 256 channels do not fit the pipelined kernels' resident weights: other kernels take the layer
    "c3_256_64_fallback": (si.single_unit_net("conv", 256, 64, k=3), 9, 8, 2, 1, "mse", ()),
    # dense 3x3, stride 2, even and odd maps
    "c3_s2_128_128": (si.single_unit_net("conv", 128, 128, k=3, stride=2), 28, 28, 3, 1, "mse", C3[:2]),
    "c3_s2_128_128_bn_odd": (si.single_unit_net("conv", 128, 128, k=3, stride=2, bn=True), 15, 13, 3, 2, "mse", C3[:2]),
    "c3_s2_64_64_odd": (si.single_unit_net("conv", 64, 64, k=3, stride=2), 11, 14, 2, 1, "mse", C3[:2]),
    # the 3-channel stem (explicit im2col + pointwise pipelines)
    "stem_3_32_s2_bn": (si.single_unit_net("conv", 3, 32, k=3, stride=2, bn=True), 63, 65, 3, 2, "mse", ("conv_im2col",) + PW[:1] + PW[2:]),
    "stem_3_32_s1": (si.single_unit_net("conv", 3, 32, k=3), 33, 31, 2, 1, "mse", ("conv_im2col",) + PW[:1] + PW[2:]),
    # depthwise 3x3
    "dw_144_s1": (si.single_unit_net("dwconv", 144, 144), 57, 56, 3, 2, "mse", DW),
    "dw_144_s1_bn": (si.single_unit_net("dwconv", 144, 144, bn=True), 56, 56, 3, 2, "mse", DW),
    "dw_192_s1_28": (si.single_unit_net("dwconv", 192, 192), 28, 28, 3, 1, "mse", DW),
    "dw_144_s2": (si.single_unit_net("dwconv", 144, 144, stride=2), 56, 56, 3, 2, "mse", DW),
    "dw_96_s2_bn_odd": (si.single_unit_net("dwconv", 96, 96, stride=2, bn=True), 31, 29, 3, 1, "mse", DW),
    "dw_960_7": (si.single_unit_net("dwconv", 960, 960, bn=True), 7, 7, 4, 1, "mse", DW),
    # depthwise 5x5 / 7x7 (EfficientNet), stride 1 and 2, even and odd maps
    "dw5_144_s1": (si.single_unit_net("dwconv", 144, 144, k=5), 29, 27, 3, 2, "mse", DW),
    "dw5_240_s2_bn_odd": (si.single_unit_net("dwconv", 240, 240, k=5, stride=2, bn=True), 31, 29, 3, 1, "mse", DW),
    "dw5_144_s2_even": (si.single_unit_net("dwconv", 144, 144, k=5, stride=2), 56, 56, 2, 1, "mse", DW),
    "dw7_48_s1_bn": (si.single_unit_net("dwconv", 48, 48, k=7, bn=True), 17, 19, 2, 2, "mse", DW),
    "dw7_48_s2_odd": (si.single_unit_net("dwconv", 48, 48, k=7, stride=2), 15, 13, 2, 1, "mse", DW),
    "dw5_16_map_smaller_than_the_kernel": (si.single_unit_net("dwconv", 16, 16, k=5, bn=True), 3, 2, 4, 2, "mse", DW),
    "dw5_16_s2_map_smaller_than_the_kernel": (si.single_unit_net("dwconv", 16, 16, k=5, stride=2), 2, 3, 4, 1, "mse", DW),
    # SiLU and squeeze-excite are smooth: held to the contract like the activation-free paths
    "pw_24_144_bn_silu": (si.single_unit_net("conv", 24, 144, bn=True, act="silu"), 29, 27, 3, 2, "mse", PW + ("silu",)),
    "pw_3_6_silu_narrow": (si.single_unit_net("conv", 3, 6, act="silu"), 9, 7, 3, 1, "mse", ("silu",)),
    "pw_24_144_bn_se": (si.single_unit_net("conv", 24, 144, bn=True, se=6), 29, 27, 3, 2, "mse", PW + ("squeeze_excite",)),
    "pw_16_240_se10_odd": (si.single_unit_net("conv", 16, 240, se=10), 7, 5, 5, 1, "mse", PW + ("squeeze_excite",)),
    "pw_3_6_se_narrow": (si.single_unit_net("conv", 3, 6, se=2), 9, 7, 3, 1, "mse", ("squeeze_excite",)),
    "dw5_144_bn_silu_se": (si.single_unit_net("dwconv", 144, 144, k=5, bn=True, act="silu", se=6), 28, 28, 3, 1, "mse", DW + ("silu", "squeeze_excite")),
    # classifier head: pool, linear, softmax cross-entropy (with and without a conv + BatchNorm in front)
    "head_1280_1000": (si.head_net(1280, 1000), 7, 7, 16, 2, "xent", ("gap_fwd", "loss_softmax_xent") + PW),
    "head_320_1280_bn_1000": (si.head_net(320, 1000, bn_conv=1280), 7, 7, 16, 1, "xent", ("gap_fwd", "loss_softmax_xent") + PW),
    "head_64_10": (si.head_net(64, 10), 5, 3, 3, 2, "xent", ("gap_fwd", "loss_softmax_xent")),
}


@pytest.mark.parametrize("bf16", [True, False], ids=["bf16", "f32"])
@pytest.mark.parametrize("name", list(CASES))
def test_kernel_path_meets_the_contract_against_the_plain_oracle(name, bf16):
    import paper_2408_08015_b200 as P
    net, h, w, B, M, loss, kernels = CASES[name]
    first, last = 0, len(net) - 1
    xs, tg, params, _ = make_inputs(net, first, last, h, w, B, M, loss, 11, bf16)
    params = si.randomize_bn(params, net, first, last, 11)       # gamma != 1, beta != 0
    plain = oracle_round(net, first, last, B, M, loss, xs, tg, params)
    P.asteroid_trace_start()
    try:
        gpu = gpu_round(net, first, last, h, w, B, M, loss, xs, tg, params, bf16)
    finally:
        ran = {k["name"] for k in P.asteroid_trace_stop()}
    if bf16:
        assert set(kernels) <= ran, "expected kernels %s, trace has %s" % (kernels, sorted(ran))
    r = compare(gpu, plain, net, first, last, 2e-2 if bf16 else 1e-4, allow=(CONTRACT,), case="kernel/%s/%s" % (name, "bf16" if bf16 else "f32"))
    print(name, summary(r))
    assert r["counts"]["mirror"] == 0 and r["counts"]["calibrated"] == 0


# ---------------------------------------------------------------------------------------------------------------------
# Every distinct conv -> BatchNorm -> activation unit of the MobileNetV2 stage, the full MobileNetV2 and the ResNet-50
# stage, each as a stage of its own at its full-size shape (so that every launcher branch the benchmarked workloads
# take - one or two operand stages, resident or streamed 3x3 weights, stride-2 3x3, im2col stem, 512-channel
# pointwise - is held to the tolerance by itself, not only inside a deep stage).  The stage output and the loss must meet
# the contract against the plain oracle.  With an activation in the unit the gradients are compared with the oracle
# that takes the masks on the stored (rounded) values; without one, with the plain oracle.
#   (kind, c_in, c_out, k, stride, h, w, micro-batch, activation)
UNITS = {
    "c2_expand_24_144_56": ("conv", 24, 144, 1, 1, 56, 56, 32, "relu6"),
    "c2_dw_144_s1_56": ("dwconv", 144, 144, 3, 1, 56, 56, 32, "relu6"),
    "c2_project_144_24_56": ("conv", 144, 24, 1, 1, 56, 56, 32, None),
    "c2_dw_144_s2_56": ("dwconv", 144, 144, 3, 2, 56, 56, 32, "relu6"),
    "c2_project_144_32_28": ("conv", 144, 32, 1, 1, 28, 28, 32, None),
    "c2_expand_32_192_28": ("conv", 32, 192, 1, 1, 28, 28, 32, "relu6"),
    "c2_dw_192_s1_28": ("dwconv", 192, 192, 3, 1, 28, 28, 32, "relu6"),
    "c2_project_192_32_28": ("conv", 192, 32, 1, 1, 28, 28, 32, None),
    "c4_pw_64_64_56": ("conv", 64, 64, 1, 1, 56, 56, 16, "relu"),
    "c4_c3_64_64_56": ("conv", 64, 64, 3, 1, 56, 56, 16, "relu"),
    "c4_pw_64_256_56": ("conv", 64, 256, 1, 1, 56, 56, 16, None),
    "c4_pw_256_64_56": ("conv", 256, 64, 1, 1, 56, 56, 16, "relu"),
    "c4_pw_256_128_56": ("conv", 256, 128, 1, 1, 56, 56, 16, "relu"),
    "c4_c3_128_128_s2_56": ("conv", 128, 128, 3, 2, 56, 56, 16, "relu"),
    "c4_pw_128_512_28": ("conv", 128, 512, 1, 1, 28, 28, 16, None),
    "c4_pw_256_512_s2_56": ("conv", 256, 512, 1, 2, 56, 56, 16, None),
    "c4_pw_512_128_28": ("conv", 512, 128, 1, 1, 28, 28, 16, "relu"),
    "c4_c3_128_128_28": ("conv", 128, 128, 3, 1, 28, 28, 16, "relu"),
    "c3_stem_3_32_s2_224": ("conv", 3, 32, 3, 2, 224, 224, 16, "relu6"),
    "c3_dw_32_s1_112": ("dwconv", 32, 32, 3, 1, 112, 112, 16, "relu6"),
    "c3_project_32_16_112": ("conv", 32, 16, 1, 1, 112, 112, 16, None),
    "c3_expand_16_96_112": ("conv", 16, 96, 1, 1, 112, 112, 16, "relu6"),
    "c3_dw_96_s2_112": ("dwconv", 96, 96, 3, 2, 112, 112, 16, "relu6"),
    "c3_expand_64_384_14": ("conv", 64, 384, 1, 1, 14, 14, 16, "relu6"),
    "c3_dw_384_s1_14": ("dwconv", 384, 384, 3, 1, 14, 14, 16, "relu6"),
    "c3_project_384_96_14": ("conv", 384, 96, 1, 1, 14, 14, 16, None),
    "c3_dw_576_s2_14": ("dwconv", 576, 576, 3, 2, 14, 14, 16, "relu6"),
    "c3_project_576_160_7": ("conv", 576, 160, 1, 1, 7, 7, 16, None),
    "c3_expand_160_960_7": ("conv", 160, 960, 1, 1, 7, 7, 16, "relu6"),
    "c3_dw_960_s1_7": ("dwconv", 960, 960, 3, 1, 7, 7, 16, "relu6"),
    "c3_project_960_320_7": ("conv", 960, 320, 1, 1, 7, 7, 16, None),
    "c3_head_320_1280_7": ("conv", 320, 1280, 1, 1, 7, 7, 16, "relu6"),
}


@pytest.mark.parametrize("name", list(UNITS))
def test_full_size_unit_bf16(name):
    kind, ci, co, k, stride, h, w, B, act = UNITS[name]
    net = si.single_unit_net(kind, ci, co, k=k, stride=stride, bn=True, act=act)
    first, last = 0, len(net) - 1
    xs, tg, params, _ = make_inputs(net, first, last, h, w, B, 1, "mse", 13, True)
    params = si.randomize_bn(params, net, first, last, 13)
    plain = oracle_round(net, first, last, B, 1, "mse", xs, tg, params)
    mirror = oracle_round(net, first, last, B, 1, "mse", xs, tg, params, store=bf16_store) if act else None
    gpu = gpu_round(net, first, last, h, w, B, 1, "mse", xs, tg, params, True)
    r = compare(gpu, plain, net, first, last, 2e-2, mirror=mirror, allow=(CONTRACT, MIRROR) if act else (CONTRACT,), outlier_frac=1e-4,
                case="unit/%s" % name)
    print(name, summary(r))
    assert r["counts"]["calibrated"] == 0
