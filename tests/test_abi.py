"""The C-ABI library loads without a GPU, exports what include/mixdq.h declares, and its
host-side argument checks answer before anything is launched."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2405_17873_b200 import build, mixdq
    build.build()
    return mixdq.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "mixdq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mixdq_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2405_17873_b200 import mixdq
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(mixdq.EXPORTS) == names


def test_no_link_time_dependency_on_the_driver():
    import subprocess
    from paper_2405_17873_b200 import mixdq
    out = subprocess.run(["ldd", mixdq.LIB_PATH], capture_output=True, text=True).stdout
    assert "libcuda.so" not in out and "libtorch" not in out


def test_version_and_strerror(lib):
    assert lib.mixdq_version() >= 100
    assert lib.mixdq_strerror(0) == b"success"
    for code in range(-6, 0):
        assert lib.mixdq_strerror(code) not in (b"", b"unknown error")
    assert lib.mixdq_strerror(-99) == b"unknown error"


def test_packed_bytes_size_laws(lib):
    out = C.c_size_t(0)
    for N, K in ((320, 320), (1280, 320), (7, 77), (640, 2048)):
        for bits, canon in ((8, K), (4, (K + 1) // 2), (3, ((K + 31) // 32) * 12)):
            assert lib.mixdq_packed_bytes(N, K, bits, 0, C.byref(out)) == 0
            assert out.value == N * canon
            assert lib.mixdq_packed_bytes(N, K, bits, 1, C.byref(out)) == 0
            assert out.value >= N * canon and out.value % 16 == 0
    # multiples of 128 codes pack without padding in the device layout too
    for bits in (3, 4, 8):
        lib.mixdq_packed_bytes(64, 1280, bits, 1, C.byref(out))
        assert out.value == 64 * 1280 * bits // 8
    assert lib.mixdq_packed_bytes(4, 4, 5, 0, C.byref(out)) == -2
    assert lib.mixdq_packed_bytes(0, 4, 4, 0, C.byref(out)) == -1
    assert lib.mixdq_packed_bytes(4, 4, 4, 7, C.byref(out)) == -1
    assert lib.mixdq_packed_bytes(4, 4, 4, 0, None) == -1


def test_argument_errors_come_back_before_any_launch(lib):
    out = C.c_size_t(0)
    assert lib.mixdq_workspace_bytes(256, 320, 320, 8, 8, C.byref(out)) == 0 and out.value > 0
    # weight-only layers: room for the fp16 expansion of the weights from 256 rows on, none below
    assert lib.mixdq_workspace_bytes(256, 320, 320, 4, 16, C.byref(out)) == 0 and out.value == 320 * 320 * 2
    assert lib.mixdq_workspace_bytes(16, 320, 320, 4, 16, C.byref(out)) == 0 and out.value == 0
    assert lib.mixdq_workspace_bytes(256, 320, 320, 5, 8, C.byref(out)) == -2
    assert lib.mixdq_workspace_bytes(0, 320, 320, 8, 8, C.byref(out)) == -1
    null = None
    fake = C.c_void_p(0x1000)       # never dereferenced: the checks below fail first
    odd = C.c_void_p(0x1008)
    # NULL tensors
    assert lib.mixdq_linear(null, 4, 32, 32, fake, 16, 8, fake, null, 8, fake, null, fake, null, 0, null, null) == -1
    assert lib.mixdq_linear(fake, 4, 32, 32, fake, 16, 8, fake, null, 8, fake, null, null, null, 0, null, null) == -1
    # row stride smaller than K, non-positive sizes
    assert lib.mixdq_linear(fake, 4, 32, 16, fake, 16, 8, fake, null, 8, fake, null, fake, null, 0, null, null) == -1
    assert lib.mixdq_linear(fake, 0, 32, 32, fake, 16, 8, fake, null, 8, fake, null, fake, null, 0, null, null) == -1
    # widths: 3-bit weights with int8 activations, asymmetric weights on the int8 path, 5-bit
    assert lib.mixdq_linear(fake, 4, 32, 32, fake, 16, 3, fake, null, 8, fake, null, fake, null, 0, null, null) == -2
    assert lib.mixdq_linear(fake, 4, 32, 32, fake, 16, 8, fake, fake, 8, fake, null, fake, null, 0, null, null) == -2
    assert lib.mixdq_linear(fake, 4, 32, 32, fake, 16, 5, fake, fake, 16, null, null, fake, null, 0, null, null) == -2
    assert lib.mixdq_linear(fake, 4, 32, 32, fake, 16, 8, fake, null, 12, fake, null, fake, null, 0, null, null) == -2
    # misaligned packed weights
    assert lib.mixdq_linear(fake, 4, 32, 32, odd, 16, 8, fake, null, 8, fake, null, fake, null, 0, null, null) == -3
    # conv stride, BOS call without the stored row
    assert lib.mixdq_conv3x3(fake, 1, 8, 8, 16, fake, 16, 3, 8, fake, null, 8, fake, null, fake, null, 0, null, null) == -1
    assert lib.mixdq_crossattn_kv(fake, 1, 2048, fake, 640, 8, fake, fake, null, fake, null, 0, null, null) == -1
    assert lib.mixdq_pack_weights(fake, 4, 32, 3, fake, null, 1, fake, null) == -2
    assert lib.mixdq_pack_weights(fake, 4, 32, 4, fake, null, 1, odd, null) == -3


def test_split_and_q8_argument_errors_come_back_before_any_launch(lib):
    out = C.c_size_t(0)
    null = None
    fake = C.c_void_p(0x1000)       # never dereferenced: the checks below fail first
    odd = C.c_void_p(0x1008)
    # scratch of a shortcut-split layer: two int8 copies + the first branch's int32 sums, each rounded up to 256 bytes
    assert lib.mixdq_split_workspace_bytes(64, 96, 32, 64, 48, C.byref(out)) == 0
    assert out.value == 64 * 32 + 64 * 64 + 64 * 48 * 4
    assert lib.mixdq_split_workspace_bytes(64, 96, 96, 64, 48, C.byref(out)) == -1    # nothing on the hi side
    assert lib.mixdq_split_workspace_bytes(64, 96, 0, 64, 48, C.byref(out)) == -1
    assert lib.mixdq_split_workspace_bytes(64, 96, 32, 64, 48, None) == -1
    big = C.c_size_t(1 << 30)
    split = lambda *a: lib.mixdq_linear_a8_split(*a)
    #            X     M   K   ldx at  Wlo   Whi   N   b  ws    slo   shi   bias  Y     wsp   bytes st    stream
    assert split(null, 64, 96, 96, 32, fake, fake, 48, 8, fake, fake, fake, null, fake, fake, big, null, null) == -1
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 8, fake, fake, fake, null, null, fake, big, null, null) == -1
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 8, fake, null, fake, null, fake, fake, big, null, null) == -1
    assert split(fake, 64, 96, 96, 96, fake, fake, 48, 8, fake, fake, fake, null, fake, fake, big, null, null) == -1
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 3, fake, fake, fake, null, fake, fake, big, null, null) == -2
    assert split(fake, 64, 96, 96, 24, fake, fake, 48, 8, fake, fake, fake, null, fake, fake, big, null, null) == -2
    assert split(fake, 64, 96, 96, 32, odd, fake, 48, 8, fake, fake, fake, null, fake, fake, big, null, null) == -3
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 8, fake, fake, fake, null, fake, odd, big, null, null) == -3
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 8, fake, fake, fake, null, fake, null, big, null, null) == -4
    assert split(fake, 64, 96, 96, 32, fake, fake, 48, 8, fake, fake, fake, null, fake, fake, 100, null, null) == -4
    conv = lambda *a: lib.mixdq_conv3x3_a8_split(*a)
    #           X     B  H  W  Cin at  Wlo   Whi   Co  s  b  ws    slo   shi   bias  Y     wsp   bytes st    stream
    assert conv(fake, 1, 8, 8, 64, 32, fake, fake, 16, 3, 8, fake, fake, fake, null, fake, fake, big, null, null) == -1
    assert conv(fake, 1, 8, 8, 64, 16, fake, fake, 16, 1, 8, fake, fake, fake, null, fake, fake, big, null, null) == -2
    assert conv(fake, 1, 6, 6, 64, 32, fake, fake, 16, 1, 8, fake, fake, fake, null, fake, fake, big, null, null) == -2
    # int8 activations kept between layers
    assert lib.mixdq_quantize_acts(null, 4, 32, 32, fake, fake, null) == -1
    assert lib.mixdq_quantize_acts(fake, 4, 32, 16, fake, fake, null) == -1       # row stride below K
    assert lib.mixdq_quantize_acts(fake, 4, 40, 40, fake, fake, null) == -2       # K % 16
    assert lib.mixdq_quantize_acts(fake, 4, 32, 32, fake, odd, null) == -3
    assert lib.mixdq_linear_q8(null, 4, 32, fake, 16, 8, fake, fake, null, fake, null, null) == -1
    assert lib.mixdq_linear_q8(fake, 4, 32, fake, 16, 8, fake, null, null, fake, null, null) == -1   # no scale
    assert lib.mixdq_linear_q8(fake, 4, 32, fake, 16, 3, fake, fake, null, fake, null, null) == -2
    assert lib.mixdq_linear_q8(fake, 4, 40, fake, 16, 8, fake, fake, null, fake, null, null) == -2
    assert lib.mixdq_linear_q8(odd, 4, 32, fake, 16, 8, fake, fake, null, fake, null, null) == -3
    assert lib.mixdq_linear_q8_acc_i32(fake, 4, 32, fake, 16, 8, null, null, null) == -1
    #                          Xq    B  H  W  Cin Wp    Co  s  b  ws    sx    bias  Y     st    stream
    assert lib.mixdq_conv3x3_q8(null, 1, 8, 8, 32, fake, 16, 1, 8, fake, fake, null, fake, null, null) == -1
    assert lib.mixdq_conv3x3_q8(fake, 1, 8, 8, 32, fake, 16, 3, 8, fake, fake, null, fake, null, null) == -1
    assert lib.mixdq_conv3x3_q8(fake, 1, 8, 8, 32, fake, 16, 1, 3, fake, fake, null, fake, null, null) == -2
    assert lib.mixdq_conv3x3_q8(fake, 1, 8, 8, 20, fake, 16, 1, 8, fake, fake, null, fake, null, null) == -2
    assert lib.mixdq_conv3x3_q8(fake, 1, 6, 6, 32, fake, 16, 1, 8, fake, fake, null, fake, null, null) == -2
    assert lib.mixdq_conv3x3_q8(odd, 1, 8, 8, 32, fake, 16, 1, 8, fake, fake, null, fake, null, null) == -3


def test_census_helpers_for_split_and_shared_quantization():
    from paper_2405_17873_b200 import synth
    layers = synth.unet_layers()
    split = {l.name: synth.shortcut_split_at(l) for l in layers if synth.shortcut_split_at(l)}
    # the nine concatenation-fed resnets of the up path (3 per level), each with its 3x3 and its 1x1 shortcut conv
    assert len(split) == 18
    assert split["res16_2560_1280#0"] == 1280 and split["res16_1920_1280#0"] == 1280
    assert split["res32_1920_640#0"] == 1280 and split["res32_1280_640#0"] == 640 and split["res32_960_640#0"] == 640
    assert split["res64_960_320#0"] == 640 and split["res64_640_320#1"] == 320 and split["sc64_640#0"] == 320
    for l in layers:
        s = synth.shortcut_split_at(l)
        assert s == 0 or (0 < s < l.Cin and s % 32 == 0 and (l.Cin - s) % 32 == 0)
    # down-path resnets widen their input, the upsampler convs keep it: never split
    assert not any(synth.shortcut_split_at(l) for l in layers if l.Cin <= l.N)
    roles = [synth.self_attention_role(l) for l in layers]
    assert roles.count(0) == roles.count(1) == roles.count(2) == 70     # 60 + 10 transformer blocks
    by_name = {l.name: synth.self_attention_role(l) for l in layers}
    assert [by_name[f"attn_1280#{i}"] for i in range(8)] == [0, 1, 2, -1, -1, -1, 0, 1]
    assert by_name["attn_1280#360"] == -1 and by_name["attn_640#60"] == -1     # proj_in / proj_out
    assert by_name["ffn1_1280#0"] == -1 and by_name["kv_1280#0"] == -1
