"""Host-side checks of the C-ABI boundary that need no GPU: the library builds, loads,
exports every symbol the header declares, and rejects bad arguments before touching CUDA."""
import ctypes
import os
import re

import pytest

import paper_2407_12077_b200 as gf

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "gf_wkv6.h")


def declared_symbols():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"GF_API[^;(]*?\b(gf_\w+)\s*\(", src)))


def test_header_declares_the_three_named_entry_points():
    names = declared_symbols()
    for must in ("gf_wkv6_prefill", "gf_wkv6_prefill_varlen", "gf_wkv6_step"):
        assert must in names


def test_library_exports_every_declared_symbol():
    gf.load_library()
    raw = ctypes.CDLL(gf.library_path())
    names = declared_symbols()
    assert len(names) >= 13
    for name in names:
        assert hasattr(raw, name), f"{name} declared in gf_wkv6.h but not exported"
    # and the binding mirrors exactly the declared set
    assert sorted(gf._SIGNATURES) == names


def test_version_and_status_strings():
    assert gf.version() >= 100
    assert gf.status_string(0) == "ok"
    seen = {gf.status_string(i) for i in range(6)}
    assert len(seen) == 6


def _call(name, *args):
    return getattr(gf.load_library(), name)(*args)


A = 0x1000  # a fake, 16-byte aligned, never dereferenced "device pointer"


def test_rejects_bad_arguments_before_any_launch():
    ptrs = [A] * 8
    # head size other than 64
    assert _call("gf_wkv6_prefill", *ptrs, 1, 8, 1, 32, None) == 2
    assert _call("gf_wkv6_step", *ptrs, 1, 1, 128, None) == 2
    assert _call("gf_wkv6_prefill_varlen", *ptrs, A, 1, 8, 8, 1, 48, None) == 2
    # negative sizes
    assert _call("gf_wkv6_prefill", *ptrs, -1, 8, 1, 64, None) == 1
    assert _call("gf_wkv6_prefill_f32", *ptrs, 1, -8, 1, 64, None) == 1
    assert _call("gf_wkv6_step_f32", *ptrs, 1, -1, 64, None) == 1
    # NULL required pointer, misaligned pointer, y aliasing an input
    for bad in (0, 3, 7):
        p = list(ptrs)
        p[bad] = None
        assert _call("gf_wkv6_prefill", *p, 1, 8, 1, 64, None) == 1
    p = list(ptrs)
    p[1] = A + 2
    assert _call("gf_wkv6_prefill", *p, 1, 8, 1, 64, None) == 1
    p = [A + 0x100 * i for i in range(8)]
    p[7] = p[2]
    assert _call("gf_wkv6_prefill", *p, 1, 8, 1, 64, None) == 1
    # varlen without cu_seqlens
    assert _call("gf_wkv6_prefill_varlen", *ptrs, None, 2, 8, 8, 1, 64, None) == 1
    # empty problems are legal no-ops that never reach CUDA
    assert _call("gf_wkv6_prefill", *ptrs, 0, 8, 1, 64, None) == 0
    assert _call("gf_wkv6_step", *ptrs, 0, 4, 64, None) == 0
    assert _call("gf_wkv6_prefill_varlen", *ptrs, A, 0, 0, 0, 4, 64, None) == 0


def test_host_entry_point_checks_workspace():
    need = gf.host_workspace_bytes(2, 128, 4, 64)
    tok = 2 * 128 * 4 * 64 * 2
    assert need >= 5 * tok + 4 * 64 * 4 + 2 * 2 * 4 * 64 * 64 * 4
    ptrs = [A] * 8
    assert _call("gf_wkv6_prefill_host", *ptrs, 2, 128, 4, 64, 0x10000, need - 1, None) == 4
    assert _call("gf_wkv6_prefill_host", *ptrs, 2, 128, 4, 64, None, need, None) == 1
    assert _call("gf_wkv6_prefill_host", *ptrs, 2, 128, 4, 32, 0x10000, need, None) == 2


def test_kernel_selector_validation():
    assert _call("gf_wkv6_set_kernel", 7) == 2
    assert _call("gf_wkv6_set_kernel", gf.KERNEL_AUTO) == 0


def test_binding_refuses_cpu_tensors():
    import torch
    t = torch.zeros((1, 4, 1, 64), dtype=torch.bfloat16)
    u = torch.zeros((1, 64))
    with pytest.raises(ValueError):
        gf.prefill(t, t, t, t, u, y=t.clone(), state_out=torch.zeros(1, 1, 64, 64))


def test_later_entry_points_reject_bad_arguments_before_any_launch():
    ptrs = [A + 0x100 * i for i in range(8)]
    for name in ("gf_wkv6_prefill_c2", "gf_wkv6_prefill_static"):
        assert _call(name, *ptrs, 1, 8, 1, 32, None) == 2                     # head size
        assert _call(name, *ptrs, -1, 8, 1, 64, None) == 1                    # negative size
        assert _call(name, *ptrs, 0, 8, 1, 64, None) == 0                     # empty: legal no-op
        p = list(ptrs); p[0] = None
        assert _call(name, *p, 1, 8, 1, 64, None) == 1                        # NULL r
        p = list(ptrs); p[7] = p[1]
        assert _call(name, *p, 1, 8, 1, 64, None) == 1                        # y aliases k
    p = list(ptrs); p[4] = A + 2
    assert _call("gf_wkv6_prefill_c2", *p, 1, 8, 1, 64, None) == 1            # misaligned u2
    assert _call("gf_wkv6_prefill_varlen_c2", *ptrs, None, 2, 8, 8, 1, 64, None) == 1
    assert _call("gf_wkv6_prefill_varlen_c2", *ptrs, A, 0, 0, 0, 4, 64, None) == 0
    assert _call("gf_wkv6_step_c2", *ptrs, 1, 1, 128, None) == 2
    assert _call("gf_wkv6_step_c2", *ptrs, 0, 4, 64, None) == 0
    # summaries
    assert _call("gf_wkv6_sequence_summary", A, A, A, A, 1, 8, 1, 32, 0, None) == 2
    assert _call("gf_wkv6_sequence_summary", A, A, A, None, 1, 8, 1, 64, 0, None) == 1
    assert _call("gf_wkv6_sequence_summary", A, A, A, A, 1, 0, 1, 64, 0, None) == 1      # a summary of nothing is not defined here
    assert _call("gf_wkv6_fold_summaries", None, None, 2, 1, 1, 64, A, None) == 1
    assert _call("gf_wkv6_fold_summaries", None, A, -1, 1, 1, 64, A, None) == 1
    assert _call("gf_wkv6_fold_summaries", None, A, 1, 0, 1, 64, A, None) == 0
    # workspace registration
    assert _call("gf_wkv6_set_workspace", A + 8, 1 << 20) == 1                # not 256-byte aligned
    assert _call("gf_wkv6_set_workspace", None, 0) == 0
    assert gf.workspace_bytes(1, 100000, 32, 48) == 0


def test_layernorm_entry_points_validate_before_any_launch():
    f = ctypes.c_float
    for name in ("gf_c2_layernorm", "gf_c2_layernorm_f32"):
        assert _call(name, A, A, A, f(1e-5), A, 0, 32, 64, None) == 0          # no rows: no-op
        assert _call(name, A, A, A, f(1e-5), A, 4, 0, 64, None) == 0           # no channels: no-op
        assert _call(name, A, A, A, f(1e-5), A, -1, 32, 64, None) == 1
        assert _call(name, A, A, A, f(-1.0), A, 4, 32, 64, None) == 1          # negative eps
        assert _call(name, A, A, A, f(float("nan")), A, 4, 32, 64, None) == 1
        assert _call(name, None, A, A, f(1e-5), A, 4, 32, 64, None) == 1
        assert _call(name, A, A, A, f(1e-5), None, 4, 32, 64, None) == 1
        assert _call(name, A + 2, A, A, f(1e-5), A, 4, 32, 64, None) == 1      # misaligned
        assert _call(name, A, A + 4, A, f(1e-5), A, 4, 32, 64, None) == 1
        assert _call(name, A, A, A, f(1e-5), A, 4, 3, 5, None) == 2            # H*N not a multiple of 8
        assert _call(name, A, A, A, f(1e-5), A, 4, 129, 64, None) == 2         # wider than 8192 channels


def test_key_compress_entry_point_validates_before_any_launch():
    name = "gf_gold_key_compress"
    assert _call(name, A, A + 0x100, A + 0x200, 0, 2048, 128, None) == 0            # no rows: no-op
    assert _call(name, A, A + 0x100, A + 0x200, -1, 2048, 128, None) == 1
    assert _call(name, None, A + 0x100, A + 0x200, 8, 2048, 128, None) == 1
    assert _call(name, A, A + 0x100, None, 8, 2048, 128, None) == 1
    assert _call(name, A + 2, A + 0x100, A + 0x200, 8, 2048, 128, None) == 1        # misaligned
    assert _call(name, A, A + 0x100, A, 8, 2048, 128, None) == 1                    # c aliases x
    assert _call(name, A, A + 0x100, A + 0x200, 8, 2044, 128, None) == 2            # D not a multiple of 8
    assert _call(name, A, A + 0x100, A + 0x200, 8, 2048, 44, None) == 2             # Dc not a multiple of 8
    assert _call(name, A, A + 0x100, A + 0x200, 8, 8192, 512, None) == 2            # Dc beyond 256


def test_split_plan_and_the_built_in_scratch_limit():
    """Host arithmetic of the sequence split (no device needed): the plan fills the GPU, respects the scratch cap by
    taking fewer segments, and on 148 SMs the array of gf_wkv6_prefill_static holds every splitting call of up to
    64 units (32 units four ways exactly) while 65..74 units do not fit even two ways."""
    lib = gf.load_library()
    SUMMARY, STATE = (64 + 64 * 64) * 4, 64 * 64 * 4
    cap = gf.STATIC_SCRATCH_BYTES
    # the header's constant, and the layout of this header's scratch formula
    hdr = open(os.path.join(ROOT, "include", "gf_wkv6.h")).read()
    assert f"#define GF_WKV6_STATIC_SCRATCH_BYTES {cap}u" in hdr
    assert cap == 32 * (3 * SUMMARY + STATE)
    for units in range(1, 149):
        for T in (64, 1023, 1024, 4096, 16384, 131072):
            H = units if units <= 64 else units // 2 if units % 2 == 0 else units
            B = units // H
            nseg, sc, nb = gf.split_plan(B, T, H, 148)
            nchunks = -(-T // 64)
            if units * 2 > 148 or nchunks < 16:
                assert (nseg, sc, nb) == (1, 0, 0), (units, T)
                continue
            assert 2 <= nseg <= 8 and units * nseg <= 148 and sc >= 8, (units, T, nseg, sc)
            assert (nseg - 1) * sc < nchunks <= nseg * sc                      # the segments cover the sequence, none empty
            assert nb == units * ((nseg - 1) * SUMMARY + STATE)
            # under the built-in array's cap: as many segments as fit, never more than unlimited, refusal only beyond 64 units
            cseg, csc, cnb = gf.split_plan(B, T, H, 148, cap)
            if units <= 64:
                assert 2 <= cseg <= nseg and cnb <= cap and cnb == units * ((cseg - 1) * SUMMARY + STATE), (units, T)
                if nb <= cap:
                    assert (cseg, csc, cnb) == (nseg, sc, nb)
            else:
                assert (cseg, csc, cnb) == (1, 0, 0), (units, T)                # gf_wkv6_prefill_static refuses these
    assert gf.split_plan(1, 4096, 32, 148) == (4, 16, cap)                      # the long-context shape fills it exactly
    assert gf.split_plan(1, 8192, 16, 148)[0] == 8 and gf.split_plan(1, 8192, 16, 148, cap)[0] == 7
    assert gf.split_plan(2, 4096, 12, 148)[0] == 6 and gf.split_plan(2, 4096, 12, 148, cap)[0] == 5
    # argument checks
    import ctypes
    n, s, b = ctypes.c_int(), ctypes.c_int(), ctypes.c_size_t()
    assert lib.gf_wkv6_split_plan(1, 4096, 4, 32, 148, 0, ctypes.byref(n), ctypes.byref(s), ctypes.byref(b)) == 2
    assert lib.gf_wkv6_split_plan(1, 4096, 4, 64, 0, 0, ctypes.byref(n), ctypes.byref(s), ctypes.byref(b)) == 1
    assert lib.gf_wkv6_split_plan(1, 4096, 4, 64, 148, 0, None, ctypes.byref(s), ctypes.byref(b)) == 1
