"""Host-side checks of the C-ABI library that need no GPU: it loads, exports
every function the header declares, and validates arguments before touching
CUDA."""
import ctypes
import os
import re

import pytest

from paper_2604_18616_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build_cuda()
    return binding.lib()


def declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for header in sorted(os.listdir(inc)):
        if not header.endswith(".h"):
            continue
        text = open(os.path.join(inc, header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names.update(re.findall(r"\b(ave_(?:attn|gemm|moe)_\w+)\s*\(", text))
    return sorted(names)


def test_header_declares_the_expected_entry_points():
    names = declared_functions()
    for n in ("ave_attn_fwd", "ave_attn_fwd_strided", "ave_attn_fwd_varlen", "ave_attn_fwd_host", "ave_attn_host_workspace_bytes", "ave_attn_device_status",
              "ave_attn_fwd_splitkv", "ave_attn_splitkv_workspace_bytes",
              "ave_attn_launch_count", "ave_attn_strerror", "ave_attn_version", "ave_attn_last_cuda_error",
              "ave_gemm_bf16_tn", "ave_gemm_bf16_nn", "ave_moe_fused_fwd", "ave_moe_workspace_bytes",
              "ave_attn_select_kernel", "ave_attn_splitkv_default_splits", "ave_attn_selftest_wait_timeout"):
        assert n in names


def test_library_exports_every_declared_symbol(lib):
    raw = ctypes.CDLL(binding.LIB_PATH)
    for n in declared_functions():
        assert hasattr(raw, n), "libave_attn.so does not export %s" % n


def test_version_and_strerror(lib):
    assert binding.version() >= 100
    seen = set()
    for code in range(0, 12):
        msg = binding.strerror(code)
        assert msg and msg != "unknown status"
        seen.add(msg)
    assert len(seen) == 12
    assert binding.strerror(12345) == "unknown status"


def test_validation_order_before_any_cuda_call(lib):
    A = 4096  # aligned fake address: validation must reject before dereferencing anything
    f = binding.ave_attn_fwd_raw
    assert f(0, A, A, A, A, 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_NULL_POINTER
    assert f(A, A, A, A, 0, 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_NULL_POINTER
    assert f(A, A, A, A, A, 0, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, A, A, 1, 2, 2, -5, 128, 64, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, A, A, 1, 6, 4, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE      # H % Hkv
    assert f(A, A, A, A, A, 1, 2, 2, 1 << 30, 128, 64, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, A, A, 1, 2, 2, 128, 128, 100, 0, 1.0) == binding.AVE_ERR_UNSUPPORTED_D
    assert f(A, A, A, A, A, 1, 2, 2, 128, 128, 264, 0, 1.0) == binding.AVE_ERR_UNSUPPORTED_D
    assert f(A, A, A, A, A, 1, 2, 2, 128, 128, 4, 0, 1.0) == binding.AVE_ERR_UNSUPPORTED_D
    assert f(A + 8, A, A, A, A, 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_MISALIGNED
    assert f(A, A, A, A + 2, A, 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_MISALIGNED
    assert f(A, A, A, A, A + 2, 1, 2, 2, 128, 128, 64, 0, 1.0) == binding.AVE_ERR_MISALIGNED
    assert f(A, A, A, A, A, 1, 2, 2, 128, 128, 64, 0, float("inf")) == binding.AVE_ERR_BAD_SCALE
    assert f(A, A, A, A, A, 1, 2, 2, 128, 128, 64, 0, float("nan")) == binding.AVE_ERR_BAD_SCALE
    # bad D outranks misalignment, bad shape outranks bad D (order of the status codes)
    assert f(A + 8, A, A, A, A, 1, 2, 2, 128, 128, 100, 0, 1.0) == binding.AVE_ERR_UNSUPPORTED_D
    assert f(A, A, A, A, A, 1, 3, 2, 128, 128, 96, 0, 1.0) == binding.AVE_ERR_BAD_SHAPE


def test_no_silent_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    A = 4096
    st = binding.ave_attn_fwd_raw(A, A, A, A, A, 1, 2, 2, 128, 128, 64, 0, 1.0)
    assert st in (binding.AVE_ERR_CUDA, binding.AVE_ERR_UNSUPPORTED_DEVICE)
    assert binding.launch_count() == 0


def test_host_workspace_bytes(lib):
    n = binding.host_workspace_bytes(4, 32, 32, 2048, 2048, 128)
    q = 4 * 32 * 2048 * 128 * 2
    assert n == 4 * q + 4 * 32 * 2048 * 4
    assert binding.host_workspace_bytes(1, 3, 2, 8, 8, 64) == 0      # invalid shape
    assert binding.host_workspace_bytes(1, 2, 2, 8, 8, 36) == 0      # unsupported D
    assert binding.host_workspace_bytes(1, 1, 1, 1, 1, 64) == 256 * 5  # each buffer rounded up to 256 B


def test_host_entry_point_validates_workspace(lib):
    A = 4096
    L = binding.lib()
    vp = ctypes.c_void_p
    st = L.ave_attn_fwd_host(vp(A), vp(A), vp(A), vp(A), vp(A), 1, 2, 2, 128, 128, 64, 0, 1.0, vp(0), 0, vp(0))
    assert st == binding.AVE_ERR_WORKSPACE
    st = L.ave_attn_fwd_host(vp(A), vp(A), vp(A), vp(A), vp(A), 1, 2, 2, 128, 128, 64, 0, 1.0, vp(A), 16, vp(0))
    assert st == binding.AVE_ERR_WORKSPACE


def test_gemm_validation_before_any_cuda_call(lib):
    A = 4096  # aligned fake address: validation must reject before dereferencing anything
    f = binding.ave_gemm_bf16_tn_raw
    assert f(0, A, A, 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert f(A, 0, A, 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert f(A, A, 0, 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert f(A, A, A, 0, 256, 64) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, 128, -8, 64) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, 128, 256, 0) == binding.AVE_ERR_BAD_SHAPE
    assert f(A, A, A, 2 ** 21, 256, 2 ** 21) == binding.AVE_ERR_BAD_SHAPE      # M * K beyond 2^40
    assert f(A, A, A, 2 ** 20, 256, 2 ** 19) == binding.AVE_ERR_BAD_SHAPE      # 2^39 elements: byte strides reach 2^40
    assert f(A, A, A, 128, 250, 64) == binding.AVE_ERR_MISALIGNED               # N not a multiple of 8
    assert f(A, A, A, 128, 256, 68) == binding.AVE_ERR_MISALIGNED               # K not a multiple of 8
    assert f(A + 8, A, A, 128, 256, 64) == binding.AVE_ERR_MISALIGNED
    g = binding.ave_gemm_bf16_nn_raw
    assert g(A, 0, A, 128, 256, 64) == binding.AVE_ERR_NULL_POINTER
    assert g(A, A, A, 128, 0, 64) == binding.AVE_ERR_BAD_SHAPE
    assert g(A, A, A, 128, 250, 64) == binding.AVE_ERR_MISALIGNED
    assert g(A, A, A + 4, 128, 256, 64) == binding.AVE_ERR_MISALIGNED


def test_register_split_guard(lib):
    """The softmax warps' setmaxnreg.inc can only draw on threads x registers-at-launch; an image
    compiled with fewer registers must be refused (128 x 64 + 256 x 216 = 63488 <= 384 x regs)."""
    assert binding.selftest_register_split(168) == binding.AVE_OK
    assert binding.selftest_register_split(166) == binding.AVE_OK
    assert binding.selftest_register_split(165) == binding.AVE_ERR_KERNEL_IMAGE
    assert binding.selftest_register_split(128) == binding.AVE_ERR_KERNEL_IMAGE
    assert "register" in binding.strerror(binding.AVE_ERR_KERNEL_IMAGE)


def test_build_checks_the_ptxas_register_report():
    ok = ("ptxas info    : Compiling entry function '_ZN3ave18attn_fwd_ws_kernelILi128ELb1ELb0ELb0EEEvx' for 'sm_100a'\n"
          "ptxas info    : Used 168 registers, used 1 barriers, 240 bytes smem\n"
          "ptxas info    : Compiling entry function '_ZN3ave16gemm_bf16_kernelILi256ELb0EEEvx' for 'sm_100a'\n"
          "ptxas info    : Used 94 registers, used 1 barriers\n")
    regs = build.kernel_registers(ok)
    assert sorted(regs.values()) == [94, 168]
    assert list(build.check_register_split(ok).values()) == [168]       # the GEMM kernel has no register split
    with pytest.raises(RuntimeError, match="registers per thread"):
        build.check_register_split(ok.replace("Used 168", "Used 160"))
    with pytest.raises(RuntimeError, match="no attention kernel"):
        build.check_register_split("")
    # the constants mirror the kernel's configuration
    src = open(os.path.join(ROOT, "paper_2604_18616_b200", "csrc", "attn_fwd_ws.cuh")).read()
    assert "kThreads = %d" % build.ATTN_THREADS in src
    assert "kRegsLight = 64" in src and "kRegsSoftmax = 216" in src
    assert build.ATTN_REGS_NEEDED == 128 * 64 + 256 * 216


def test_selftest_hooks_validate_their_arguments(lib):
    assert binding.selftest_inject_failures(3, 1) == binding.AVE_ERR_BAD_SHAPE
    assert binding.selftest_inject_failures(binding.INJECT_LAUNCH_FAILURE, -1) == binding.AVE_ERR_BAD_SHAPE
    assert binding.selftest_inject_failures(binding.INJECT_LAUNCH_FAILURE, 0) == binding.AVE_OK
    assert binding.lib().ave_attn_selftest_wait_timeout(5, None) == binding.AVE_ERR_BAD_SHAPE
    assert binding.lib().ave_attn_selftest_wait_timeout(40, None) == binding.AVE_ERR_BAD_SHAPE
    assert binding.tensor_map_encodes() >= 0


def test_moe_validation_before_any_cuda_call(lib):
    A = 4096
    L = binding.lib()
    vp = ctypes.c_void_p
    def f(ptrs, T, C, F, E, K, ws=A, ws_bytes=1 << 40):
        return L.ave_moe_fused_fwd(*[vp(p) for p in ptrs], T, C, F, E, K, vp(ws), ctypes.c_size_t(ws_bytes), vp(0))
    ok = [A] * 9
    assert f([0] + ok[1:], 4, 256, 128, 2, 2) == binding.AVE_ERR_NULL_POINTER
    assert f(ok[:8] + [0], 4, 256, 128, 2, 2) == binding.AVE_ERR_NULL_POINTER
    assert f(ok, 0, 256, 128, 2, 2) == binding.AVE_ERR_BAD_SHAPE
    assert f(ok, 4, 250, 128, 2, 2) == binding.AVE_ERR_BAD_SHAPE          # C not a multiple of 128
    assert f(ok, 4, 256, 100, 2, 2) == binding.AVE_ERR_BAD_SHAPE          # F not a multiple of 128
    assert f(ok, 1 << 22, 256, 128, 2, 8) == binding.AVE_ERR_BAD_SHAPE    # T * K too large
    assert f([A + 8] + ok[1:], 4, 256, 128, 2, 2) == binding.AVE_ERR_MISALIGNED
    assert f(ok[:1] + [A + 2] + ok[2:], 4, 256, 128, 2, 2) == binding.AVE_ERR_MISALIGNED
    assert f(ok, 4, 256, 128, 2, 2, ws=0) == binding.AVE_ERR_WORKSPACE
    assert f(ok, 4, 256, 128, 2, 2, ws_bytes=16) == binding.AVE_ERR_WORKSPACE
    n = binding.moe_workspace_bytes(4096, 7168, 2048, 32, 4)
    rows = 128 * (4096 * 4 // 128 + 32)
    assert n >= rows * (7168 + 7168 * 4 + 2048) and n % 256 == 0
