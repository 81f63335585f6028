"""Host-side checks that need no GPU: the library loads, exports what the header declares,
and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

from paper_2606_06034_b200 import binding as gdn
from paper_2606_06034_b200 import build as gdn_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    gdn_build.build()
    return gdn.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "gdnprep.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gdn_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    names = _declared_functions()
    assert "gdn_chunk_prepare" in names and "gdn_device_status" in names
    for name in names:
        assert hasattr(lib, name), name
    assert set(names) == set(gdn.EXPORTS)


def test_defaults_follow_the_paper(lib):
    assert [lib.gdn_default_order(c) for c in (16, 32, 64, 128)] == [3, 3, 3, 3]
    assert [lib.gdn_default_order(c) for c in (2, 3, 4)] == [1, 2, 3]  # below the chunk size
    assert [lib.gdn_default_residual_steps(c) for c in (16, 32, 64, 128)] == [3, 4, 8, 8]


def test_int8_decay_table_matches_the_oracle(lib):
    from oracle import gdn_oracle_int8 as orq
    assert lib.gdn_int8_lut_checksum() == orq.lut_checksum()


def test_status_strings(lib):
    for code in range(0, -9, -1):
        assert lib.gdn_status_string(code)
    assert gdn.status_string(gdn.GDN_ERR_TIMEOUT).startswith("bounded wait")


def test_bad_arguments_are_rejected_without_a_device(lib):
    buf = ctypes.create_string_buffer(4096)
    base = ctypes.addressof(buf)
    base += (-base) % 16
    p = ctypes.c_void_p(base)
    mis = ctypes.c_void_p(base + 4)

    def call(K=p, V=p, beta=p, g=p, B=1, H=1, T=128, C=64, dk=128, dv=128, N=-1, S=-1, dt=1, W=p, U=p, Ti=p):
        return lib.gdn_chunk_prepare(K, V, beta, g, B, H, T, C, dk, dv, N, S, dt, W, U, Ti, None)

    assert call(K=None) == gdn.GDN_ERR_NULL
    assert call(W=None) == gdn.GDN_ERR_NULL
    assert call(T=100) == gdn.GDN_ERR_INVALID_ARG
    assert call(C=1, T=128) == gdn.GDN_ERR_INVALID_ARG
    assert call(N=0) == gdn.GDN_ERR_INVALID_ARG
    assert call(N=64) == gdn.GDN_ERR_INVALID_ARG
    assert call(S=-2) == gdn.GDN_ERR_INVALID_ARG
    assert call(dt=7) == gdn.GDN_ERR_INVALID_ARG
    assert call(C=256, T=256) == gdn.GDN_ERR_UNSUPPORTED
    assert call(g=mis) == gdn.GDN_ERR_ALIGN
    assert call(Ti=mis) == gdn.GDN_ERR_ALIGN
    assert lib.gdn_chunk_prepare_gqa(p, p, p, p, 1, 2, 3, 128, 64, 128, 128, -1, -1, 1, p, p, p, None) == gdn.GDN_ERR_INVALID_ARG
    assert lib.gdn_chunk_prepare_fwdsubst(p, p, p, p, 1, 1, 1, 128, 64, 128, 128, 1, 5, p, p, p, None) == gdn.GDN_ERR_INVALID_ARG
    vl = lambda **kw: lib.gdn_chunk_prepare_varlen(*[kw.get(k, d) for k, d in (
        ("K", p), ("V", p), ("beta", p), ("g", p), ("cs", p), ("cl", p), ("n", 2), ("T", 128), ("Hk", 1), ("Hv", 1), ("C", 64),
        ("dk", 128), ("dv", 128), ("N", -1), ("S", -1), ("W", p), ("U", p), ("Ti", p), ("flags", 0), ("stream", None))])
    assert vl(cs=None) == gdn.GDN_ERR_NULL
    assert vl(n=-1) == gdn.GDN_ERR_INVALID_ARG
    assert vl(C=48) == gdn.GDN_ERR_UNSUPPORTED
    assert vl(flags=gdn.GDN_FLAG_OUT_FP32) == gdn.GDN_ERR_INVALID_ARG
    assert vl(Hk=2, Hv=3) == gdn.GDN_ERR_INVALID_ARG
    assert vl(W=mis) == gdn.GDN_ERR_ALIGN
    lib.gdn_chunk_state_segmented_workspace.restype = ctypes.c_size_t
    assert lib.gdn_chunk_state_segmented_workspace(32, 1) == 0
    assert lib.gdn_chunk_state_segmented_workspace(32, 3) >= (2 * 3 + 2 * 3) * 32 * 128 * 128 * 4
    seg = lambda **kw: lib.gdn_chunk_state_output_segmented(*[kw.get(k, d) for k, d in (
        ("Q", p), ("K", p), ("W", p), ("U", p), ("g", p), ("Hk", 1), ("Hv", 1), ("T", 256), ("C", 64), ("dk", 128), ("dv", 128),
        ("scale", ctypes.c_float(1.0)), ("S_in", None), ("O", p), ("S_out", None), ("segments", 2), ("ws", p),
        ("ws_bytes", ctypes.c_size_t(1 << 30)), ("flags", 0), ("stream", None))])
    assert seg(Q=None) == gdn.GDN_ERR_NULL
    assert seg(ws=None) == gdn.GDN_ERR_NULL
    assert seg(segments=0) == gdn.GDN_ERR_INVALID_ARG
    assert seg(ws_bytes=ctypes.c_size_t(16)) == gdn.GDN_ERR_INVALID_ARG
    assert seg(T=100) == gdn.GDN_ERR_INVALID_ARG
    assert seg(flags=gdn.GDN_FLAG_W_GATED) == gdn.GDN_ERR_INVALID_ARG
    assert seg(ws=mis) == gdn.GDN_ERR_ALIGN
    # the variant of the segmented call on built-in scratch: same checks, no workspace argument
    na = lambda **kw: lib.gdn_chunk_state_output_segmented_noalloc(*[kw.get(k, d) for k, d in (
        ("Q", p), ("K", p), ("W", p), ("U", p), ("g", p), ("Hk", 1), ("Hv", 1), ("T", 256), ("C", 64), ("dk", 128), ("dv", 128),
        ("scale", ctypes.c_float(1.0)), ("S_in", None), ("O", p), ("S_out", None), ("segments", 2), ("flags", 0), ("stream", None))])
    assert na(Q=None) == gdn.GDN_ERR_NULL
    assert na(segments=0) == gdn.GDN_ERR_INVALID_ARG
    assert na(T=100) == gdn.GDN_ERR_INVALID_ARG
    assert na(flags=gdn.GDN_FLAG_W_GATED) == gdn.GDN_ERR_INVALID_ARG
    assert na(O=mis) == gdn.GDN_ERR_ALIGN
    # the integer entry points
    i8 = lambda fn, **kw: fn(*[kw.get(k, d) for k, d in (
        ("Kq", p), ("Vq", p), ("ke", p), ("ve", p), ("bq", p), ("dq", p), ("B", 1), ("Hk", 1), ("Hv", 1), ("T", 128), ("C", 64),
        ("dk", 128), ("dv", 128), ("N", -1), ("S", -1), ("Wq", p), ("Uq", p), ("we", p), ("ue", p), ("Toff", p), ("te", p),
        ("dbg", None), ("stream", None))])
    for fn in (lib.gdn_chunk_prepare_int8, lib.gdn_chunk_prepare_int16):
        assert i8(fn, Kq=None) == gdn.GDN_ERR_NULL
        assert i8(fn, te=None) == gdn.GDN_ERR_NULL
        assert i8(fn, T=100) == gdn.GDN_ERR_INVALID_ARG
        assert i8(fn, Hk=2, Hv=3) == gdn.GDN_ERR_INVALID_ARG
        assert i8(fn, N=0) == gdn.GDN_ERR_INVALID_ARG
        assert i8(fn, S=-2) == gdn.GDN_ERR_INVALID_ARG
        assert i8(fn, Wq=mis) == gdn.GDN_ERR_ALIGN
        assert i8(fn, dbg=mis) == gdn.GDN_ERR_ALIGN
    # INT8 on chunks of 128 tokens: T must be a multiple of 128 (the int16 entry point has no such form)
    assert i8(lib.gdn_chunk_prepare_int8, C=128, T=192) == gdn.GDN_ERR_INVALID_ARG
    assert lib.gdn_chunk_prepare_fwdsubst(p, p, p, p, 1, 1, 1, 128, 32, 128, 128, 1, gdn.GDN_FWDSUBST_BLOCKED_TC, p, p, p, None) in (
        gdn.GDN_ERR_UNSUPPORTED,)
    assert lib.gdn_chunk_prepare_fwdsubst(p, p, p, p, 1, 1, 1, 128, 64, 128, 128, 0, gdn.GDN_FWDSUBST_BLOCKED_TC, p, p, p, None) == \
        gdn.GDN_ERR_UNSUPPORTED  # bf16 only
    # valid arguments but no sm_100 device in this process: refused, nothing launched
    import torch
    if not torch.cuda.is_available():
        assert call() == gdn.GDN_ERR_ARCH
        assert lib.gdn_launch_count() == 0


def test_binding_refuses_host_tensors():
    import torch
    K = torch.zeros(1, 1, 64, 128, dtype=torch.bfloat16)
    b = torch.zeros(1, 1, 64)
    with pytest.raises(ValueError):
        gdn.chunk_prepare(K, K, b, b, 64)


def test_chunk_table_of_packed_sequences():
    """Host-side chunking of packed sequences (each sequence chunked from its own first token, last chunk short),
    against the oracle's own table."""
    from oracle import gdn_oracle as orc
    for C in (16, 64, 128):
        for cu in ([0, 5, 5, 70, 198, 199, 327], [0, C], [0, C - 1, 2 * C], [0]):
            start, length = gdn.chunk_table(cu, C)
            o_start, o_length = orc.chunk_table(cu, C)
            assert list(start) == list(o_start) and list(length) == list(o_length)
            assert sum(length) == cu[-1] and all(1 <= n <= C for n in length)
    with pytest.raises(ValueError):
        gdn.chunk_table([0, 10, 5], 64)



def test_public_header_compiles_on_its_own_as_c_and_cpp(tmp_path):
    """include/gdnprep.h is the boundary: plain C (no torch, no CUDA headers), usable from C99 and C++."""
    import shutil
    import subprocess
    inc = os.path.join(ROOT, "include")
    for compiler, std, ext in (("gcc", "-std=c99", "c"), ("g++", "-std=c++17", "cpp")):
        if shutil.which(compiler) is None:
            pytest.skip(f"{compiler} not available")
        src = tmp_path / f"t.{ext}"
        src.write_text('#include "gdnprep.h"\nint main(void) { return gdn_default_order(64) == 0; }\n')
        r = subprocess.run([compiler, std, "-Wall", "-Wextra", "-pedantic", "-I", inc, "-c", str(src), "-o", str(tmp_path / "t.o")],
                           capture_output=True, text=True)
        assert r.returncode == 0, r.stderr


def test_hot_kernels_are_built_without_register_spills():
    """The tensor-core kernels run at the register limit of two CTAs per SM, where even 4 bytes of spill per thread
    were measured to cost 5 % (the reloads sit on a tile's dependent chain). The build keeps ptxas's resource report:
    the instantiations behind the benchmark's configurations must be free of spills."""
    from paper_2606_06034_b200 import build as gdn_build
    gdn_build.build()
    res = gdn_build.kernel_resources("chunk_tc_bf16.cu")
    # <C, NB, MODE, MERGE, EX, DBL, PERM>: the default C = 64 instantiation in both forms (M = 128 products; M = 64
    # products per chunk for large launches), the C = 128 one, C = 32 and C = 16, and the C = 64 instantiations with
    # the optional prologue / layouts (EX = 1) and for packed sequences (EX = 3)
    for key in ("chunk_tc_kernelILi64ELi3ELi0ELb0ELi0ELi8ELb0E", "chunk_tc_kernelILi64ELi3ELi0ELb0ELi0ELi8ELb1E",
                "chunk_tc_kernelILi64ELi3ELi0ELb1ELi0ELi8ELb0E",
                "chunk_tc_kernelILi32ELi3ELi0ELb0ELi0ELi0ELb0E", "chunk_tc_kernelILi16ELi3ELi0ELb0ELi0ELi0ELb0E",
                "chunk_tc_kernelILi64ELi3ELi0ELb0ELi1ELi8ELb0E", "chunk_tc_kernelILi64ELi3ELi0ELb0ELi3ELi8ELb0E"):
        hits = [v for k, v in res.items() if key in k]
        assert len(hits) == 1, key
        assert hits[0]["spill_stores"] == 0 and hits[0]["spill_loads"] == 0, (key, hits[0])
        assert hits[0]["registers"] <= 128
    res = gdn_build.kernel_resources("chunk_tc_int8.cu")
    main = [v for k, v in res.items() if "chunk_tc_int8_kernel" in k]  # with and without the accumulator dump
    assert len(main) == 2 and all(v["spill_stores"] == 0 and v["registers"] <= 128 for v in main)
    res = gdn_build.kernel_resources("chunk_state.cu")
    assert all(v["spill_stores"] == 0 for k, v in res.items() if "chunk_state_kernel" in k)
