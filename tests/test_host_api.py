"""CPU-only checks of the C-ABI library: it loads, exports every declared symbol, and its
host-side logic (argument validation, workspace sizing, split planning) behaves as declared.
No kernel is launched here."""
import ctypes
import re
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    from paper_2605_29157_b200 import build
    build.build()
    from paper_2605_29157_b200 import binding
    return binding


def test_every_declared_symbol_is_exported(lib):
    header = (ROOT / "include" / "parallax.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(parallax_\w+)\s*\(", header))
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib._lib, name), f"{name} declared in parallax.h but not exported"
    assert declared == set(lib.EXPORTS)
    hooks = re.sub(r"/\*.*?\*/", "", (ROOT / "include" / "parallax_test_hooks.h").read_text(), flags=re.S)
    declared_hooks = set(re.findall(r"\b(plx_test_\w+)\s*\(", hooks))
    assert declared_hooks == set(lib.TEST_HOOK_EXPORTS)
    for name in declared_hooks:
        assert hasattr(lib._lib, name), f"{name} declared in parallax_test_hooks.h but not exported"


def test_version_and_status_strings(lib):
    assert lib.parallax_version() >= 100
    seen = set()
    for code in range(0, -10, -1):
        s = lib.status_string(code)
        assert s and s != "unknown status" and s not in seen
        seen.add(s)
    assert lib.status_string(-99) == "unknown status"


def test_partial_stride_and_workspace_bytes(lib):
    assert lib.parallax_partial_stride(128) == 260
    assert lib.parallax_partial_stride(64) == 132
    w1 = lib.parallax_decode_workspace_bytes(8, 16, 128, 1)
    w8 = lib.parallax_decode_workspace_bytes(8, 16, 128, 8)
    assert w8 - w1 == 8 * 16 * 7 * 260 * 4
    assert w1 >= 256 + 8 * 16 * 260 * 4 + 8 * 16 * 128 * (2 + 2 + 4)
    assert lib.parallax_decode_workspace_bytes(0, 16, 128, 1) == 0
    assert lib.parallax_decode_workspace_bytes(8, 16, 128, 0) == 0
    assert lib.parallax_decode_workspace_bytes(8, 16, 128, lib.PLX_MAX_SPLITS + 1) == 0


@pytest.mark.parametrize("B,Hkv,T,ragged", [(1, 1, 512, False), (8, 8, 4096, False), (64, 8, 8192, False),
                                            (2, 8, 131072, False), (128, 8, 32768, True), (1, 1, 1, False),
                                            (3, 2, 100000, True), (2048, 8, 128, False)])
def test_plan_invariants(lib, B, Hkv, T, ragged):
    chunk, ns = lib.parallax_decode_plan(B, 2 * Hkv, Hkv, 128, T, 148, ragged)
    assert chunk % 64 == 0 and chunk > 0
    assert ns == -(-T // chunk) and 1 <= ns <= lib.PLX_MAX_SPLITS
    assert ns == 1 or chunk >= 256
    # enough CTAs to saturate HBM (~130 on a B200) whenever the context is long enough to allow it
    if T >= 148 * 2 * 256:
        assert B * Hkv * ns >= 128


def test_plan_uses_the_device_for_few_long_streams(lib):
    chunk, ns = lib.parallax_decode_plan(2, 16, 8, 128, 131072, 148, False)
    assert 128 <= 16 * ns <= 148 * 2
    chunk1, ns1 = lib.parallax_decode_plan(1, 2, 1, 64, 512, 148, False)
    assert ns1 in (1, 2)


def test_argument_validation_without_a_device(lib):
    """Every error below is detected on the host before any CUDA call."""
    L = lib._lib
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x1002)
    none = None
    args = dict(B=2, Hq=4, Hkv=2, D=128, T=64)

    def fwd(q=fake, r=fake, k=fake, v=fake, out=fake, B=2, Hq=4, Hkv=2, D=128, T=64, dt=0, ws=none, wsb=0, ns=1):
        return L.parallax_decode_fwd_ex(q, r, k, v, none, out, B, Hq, Hkv, D, T, 0.1, dt, ws, wsb, ns, none)

    assert fwd(q=none) == lib.PLX_ERR_NULL_POINTER
    assert fwd(out=none) == lib.PLX_ERR_NULL_POINTER
    assert fwd(Hq=3) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(B=0) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(T=0) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(D=96) == lib.PLX_ERR_UNSUPPORTED
    # more than 64 query heads per KV head: beyond the decode kernel (the stand-alone split kernel says so;
    # parallax_decode_fwd_ex hands such groups to the tensor-core kernel)
    assert L.parallax_decode_splitkv_partial(fake, fake, fake, fake, none, fake, 2, 260, 2, 128, 64, 0.1, 64, 1, none,
                                             none) == lib.PLX_ERR_UNSUPPORTED
    assert fwd(dt=7) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(ns=-1) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(ns=lib.PLX_MAX_SPLITS + 1) == lib.PLX_ERR_BAD_SHAPE
    assert fwd(k=odd) == lib.PLX_ERR_ALIGNMENT
    assert fwd(T=4096, ns=4) == lib.PLX_ERR_WORKSPACE                 # split without workspace
    assert fwd(T=4096, ns=4, ws=fake, wsb=1024) == lib.PLX_ERR_WORKSPACE
    assert fwd(B=1 << 20, T=1 << 20) == lib.PLX_ERR_BAD_SHAPE         # row index would overflow

    assert L.parallax_decode_fwd(fake, fake, fake, fake, none, fake, 2, 4, 2, 128, 0.1, none) in (
        lib.PLX_ERR_NEED_LAYOUT,)
    assert L.parallax_set_layout(0, 0, none, 0) == lib.PLX_ERR_BAD_SHAPE
    assert L.parallax_set_layout(64, 3, none, 0) == lib.PLX_ERR_BAD_SHAPE

    part = L.parallax_decode_splitkv_partial
    assert part(fake, fake, fake, fake, none, none, 2, 4, 2, 128, 64, 0.1, 64, 1, none, none) == lib.PLX_ERR_NULL_POINTER
    assert part(fake, fake, fake, fake, none, fake, 2, 4, 2, 128, 64, 0.1, 24, 3, none, none) == lib.PLX_ERR_BAD_SHAPE
    assert part(fake, fake, fake, fake, none, fake, 2, 4, 2, 128, 64, 0.1, 32, 1, none, none) == lib.PLX_ERR_BAD_SHAPE

    comb = L.parallax_decode_combine
    assert comb(none, none, fake, 2, 4, 128, 3, 0, none) == lib.PLX_ERR_NULL_POINTER
    assert comb(fake, none, fake, 2, 4, 96, 3, 0, none) == lib.PLX_ERR_UNSUPPORTED
    assert comb(fake, none, fake, 2, 4, 128, 0, 0, none) == lib.PLX_ERR_BAD_SHAPE
    assert comb(odd, none, fake, 2, 4, 128, 3, 0, none) == lib.PLX_ERR_ALIGNMENT

    host = L.parallax_decode_fwd_host
    assert host(none, fake, fake, fake, none, fake, 2, 4, 2, 128, 64, 0.1, 0, fake, 1 << 20, 1, none) == lib.PLX_ERR_NULL_POINTER
    assert host(fake, fake, fake, fake, none, fake, 2, 4, 2, 128, 64, 0.1, 0, none, 0, 1, none) == lib.PLX_ERR_WORKSPACE
    assert host(fake, fake, fake, fake, none, fake, 2, 4, 2, 128, 64, 0.1, 0, fake, 100, 1, none) == lib.PLX_ERR_WORKSPACE


def test_training_entry_points_validate_on_the_host(lib):
    """Saved-state forward and backward: every error below is detected before any CUDA call."""
    L = lib._lib
    fake, odd, none = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008), None

    def save(lse=fake, tbar=fake, vbar=fake, D=128, Hq=4, prec=0):
        return L.parallax_prefill_fwd_save(fake, fake, fake, fake, none, fake, lse, tbar, vbar, 2, Hq, 2, D, 64, 64, 0.1, 0,
                                           prec, none, none)

    assert save(lse=none) == lib.PLX_ERR_NULL_POINTER
    assert save(vbar=none) == lib.PLX_ERR_NULL_POINTER
    assert save(vbar=odd) == lib.PLX_ERR_ALIGNMENT
    assert save(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert save(Hq=3) == lib.PLX_ERR_BAD_SHAPE
    assert save(prec=5) == lib.PLX_ERR_BAD_SHAPE

    need = lib.parallax_prefill_bwd_workspace_bytes(2, 4, 64)
    assert need == (2 * 4 * 64 + 64) * 16
    assert lib.parallax_prefill_bwd_workspace_bytes(0, 4, 64) == 0

    def bwd(dout=fake, dk=fake, ws=fake, wsb=need, D=128, Hq=4, io=0, gd=1, Lq=64):
        return L.parallax_prefill_bwd(fake, fake, fake, fake, dout, fake, fake, fake, fake, none, fake, fake, dk, fake,
                                      2, Hq, 2, D, Lq, 64, 0.1, io, gd, ws, wsb, none, none)

    assert bwd(dout=none) == lib.PLX_ERR_NULL_POINTER
    assert bwd(ws=none) == lib.PLX_ERR_NULL_POINTER
    assert bwd(dk=odd) == lib.PLX_ERR_ALIGNMENT
    assert bwd(D=32) == lib.PLX_ERR_UNSUPPORTED
    assert bwd(Hq=5) == lib.PLX_ERR_BAD_SHAPE
    assert bwd(Lq=0) == lib.PLX_ERR_BAD_SHAPE
    assert bwd(io=3) == lib.PLX_ERR_BAD_SHAPE
    assert bwd(gd=-1) == lib.PLX_ERR_BAD_SHAPE
    assert bwd(wsb=need - 1) == lib.PLX_ERR_WORKSPACE


def test_serving_variant_entry_points_validate_on_the_host(lib):
    """e4m3-cache and paged entry points: argument errors detected before any CUDA call."""
    L = lib._lib
    fake, none = ctypes.c_void_p(0x1000), None

    def fp8(D=128, ks=0.5, vs=0.5, k=fake):
        return L.parallax_decode_fwd_fp8(fake, fake, k, fake, none, fake, 2, 4, 2, D, 64, 0.1, ks, vs, 0, none, 0, 1, none)

    assert fp8(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert fp8(ks=0.0) == lib.PLX_ERR_BAD_SHAPE
    assert fp8(vs=float("inf")) == lib.PLX_ERR_BAD_SHAPE
    assert fp8(vs=float("nan")) == lib.PLX_ERR_BAD_SHAPE
    assert fp8(k=none) == lib.PLX_ERR_NULL_POINTER

    def paged_fp8(table=fake, ps=64, ks=0.5):
        return L.parallax_decode_fwd_paged_fp8(fake, fake, fake, fake, table, none, fake, 2, 4, 2, 128, 10, ps, 4, 0.1,
                                               ks, 0.5, 0, none, 0, 1, none)

    assert paged_fp8(table=none) == lib.PLX_ERR_NULL_POINTER
    assert paged_fp8(ps=24) == lib.PLX_ERR_BAD_SHAPE
    assert paged_fp8(ks=-1.0) == lib.PLX_ERR_BAD_SHAPE

    def paged_prefill(table=fake, ps=64, prec=0, D=128):
        return L.parallax_prefill_fwd_paged(fake, fake, fake, fake, table, none, fake, 2, 4, 2, D, 16, 10, ps, 4, 0.1, 0,
                                            prec, none, none)

    assert paged_prefill(table=none) == lib.PLX_ERR_NULL_POINTER
    assert paged_prefill(ps=32) == lib.PLX_ERR_BAD_SHAPE      # a 64-key tile must not straddle a page
    assert paged_prefill(prec=9) == lib.PLX_ERR_BAD_SHAPE
    assert paged_prefill(D=96) == lib.PLX_ERR_UNSUPPORTED


def test_host_buffer_entry_refuses_a_split_count_without_room_before_staging(lib):
    """A forced split count whose records do not fit the workspace (or one outside the legal range) is
    refused by the host-buffer entry before the first copy or launch is enqueued."""
    L = lib._lib
    fake = ctypes.c_void_p(0x1000)
    B, Hq, Hkv, D, T = 2, 4, 2, 128, 8192
    small = lib.parallax_decode_workspace_bytes(B, Hq, D, 2)

    def host(ns, wsb=small):
        return L.parallax_decode_fwd_host(fake, fake, fake, fake, None, fake, B, Hq, Hkv, D, T, 0.1, 0, fake, wsb, ns, None)

    assert host(64) == lib.PLX_ERR_WORKSPACE
    assert host(-1) == lib.PLX_ERR_BAD_SHAPE
    assert host(lib.PLX_MAX_SPLITS + 1) == lib.PLX_ERR_BAD_SHAPE


def test_per_head_scale_and_one_call_step_entry_points_validate_on_the_host(lib):
    """Per-KV-head e4m3 scales and the one-call decode step: argument errors detected before any CUDA call
    (the step must not touch the cache when its attention arguments are invalid)."""
    L = lib._lib
    fake, odd, none = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1002), None

    def per_head(ks=fake, vs=fake, D=128, Hq=4):
        return L.parallax_decode_fwd_fp8_per_head(fake, fake, fake, fake, none, fake, 2, Hq, 2, D, 64, 0.1, ks, vs, 0,
                                                  none, 0, 1, none)

    assert per_head(ks=none) == lib.PLX_ERR_NULL_POINTER
    assert per_head(vs=none) == lib.PLX_ERR_NULL_POINTER
    assert per_head(ks=odd) == lib.PLX_ERR_ALIGNMENT
    assert per_head(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert per_head(Hq=5) == lib.PLX_ERR_BAD_SHAPE

    def paged_per_head(table=fake, ks=fake, ps=64):
        return L.parallax_decode_fwd_paged_fp8_per_head(fake, fake, fake, fake, table, none, fake, 2, 4, 2, 128, 10, ps,
                                                        4, 0.1, ks, fake, 0, none, 0, 1, none)

    assert paged_per_head(table=none) == lib.PLX_ERR_NULL_POINTER
    assert paged_per_head(ks=none) == lib.PLX_ERR_NULL_POINTER
    assert paged_per_head(ps=24) == lib.PLX_ERR_BAD_SHAPE

    def step(out=fake, q_out=fake, D=128, Hq=4, ns=1, out_dtype=0, T=64):
        return L.parallax_decode_step(fake, fake, fake, fake, none, none, none, none, q_out, fake, fake, fake, out, 2, Hq,
                                      2, D, T, 1e-6, 1e6, 0, 0.1, out_dtype, none, 0, ns, none)

    assert step(out=none) == lib.PLX_ERR_NULL_POINTER
    assert step(q_out=none) == lib.PLX_ERR_NULL_POINTER
    assert step(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert step(Hq=3) == lib.PLX_ERR_BAD_SHAPE
    assert step(ns=lib.PLX_MAX_SPLITS + 1) == lib.PLX_ERR_BAD_SHAPE
    assert step(out_dtype=7) == lib.PLX_ERR_BAD_SHAPE
    assert step(ns=4, T=4096) == lib.PLX_ERR_WORKSPACE   # forced splits without room for their records


def test_multi_token_decode_entry_point_validates_on_the_host(lib):
    L = lib._lib
    fake, none = ctypes.c_void_p(0x1000), None

    def multi(Lq=4, Hq=4, Hkv=2, D=128, out=fake):
        return L.parallax_decode_fwd_multi(fake, fake, fake, fake, none, out, 2, Hq, Hkv, D, Lq, 64, 0.1, 0, none, 0, 1, none)

    assert multi(Lq=0) == lib.PLX_ERR_BAD_SHAPE
    assert multi(Hq=5) == lib.PLX_ERR_BAD_SHAPE
    assert multi(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert multi(out=none) == lib.PLX_ERR_NULL_POINTER


def test_split_prefill_entry_point_validates_on_the_host(lib):
    L = lib._lib
    fake, odd, none = ctypes.c_void_p(0x1000), ctypes.c_void_p(0x1008), None
    assert lib.parallax_prefill_workspace_bytes(2, 4, 128, 64, 8) == 2 * 4 * 64 * 8 * (2 * 128 + 4) * 4
    assert lib.parallax_prefill_workspace_bytes(2, 4, 128, 0, 8) == 0
    assert lib.parallax_prefill_workspace_bytes(2, 4, 128, 64, lib.PLX_MAX_SPLITS + 1) == 0

    def ex(ws=fake, wsb=1 << 20, ns=2, D=128, out=fake):
        return L.parallax_prefill_fwd_ex(fake, fake, fake, fake, none, out, 2, 4, 2, D, 64, 4096, 0.1, 0, 0, ws, wsb, ns,
                                         none, none)

    assert ex(out=none) == lib.PLX_ERR_NULL_POINTER
    assert ex(D=96) == lib.PLX_ERR_UNSUPPORTED
    assert ex(ns=-1) == lib.PLX_ERR_BAD_SHAPE
    assert ex(ns=lib.PLX_MAX_SPLITS + 1) == lib.PLX_ERR_BAD_SHAPE
    assert ex(ws=none, wsb=0, ns=4) == lib.PLX_ERR_WORKSPACE


def test_public_header_is_plain_c():
    """The boundary is a C ABI: the header has to compile as C99 (and as C++) on its own, and the options
    struct of parallax_decode_fwd_args must have the layout the binding mirrors."""
    import shutil
    import subprocess
    hdr = str(ROOT / "include" / "parallax.h")
    if shutil.which("gcc"):
        subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only", "-x", "c", hdr],
                       check=True)
        prog = ('#include <stdio.h>\n#include <stddef.h>\n#include "parallax.h"\nint main(void){printf("%zu %zu %zu %zu",'
                'sizeof(parallax_decode_args), offsetof(parallax_decode_args, k_scale),'
                'offsetof(parallax_decode_args, block_table), offsetof(parallax_decode_args, stream));return 0;}')
        import tempfile
        with tempfile.TemporaryDirectory() as d:
            src, exe = Path(d) / "t.c", Path(d) / "t"
            src.write_text(prog)
            subprocess.run(["gcc", "-std=c99", "-I", str(ROOT / "include"), str(src), "-o", str(exe)], check=True)
            sizes = [int(v) for v in subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split()]
        from paper_2605_29157_b200 import binding
        A = binding.ParallaxDecodeArgs
        assert sizes == [ctypes.sizeof(A), A.k_scale.offset, A.block_table.offset, A.stream.offset]
    if shutil.which("g++"):
        subprocess.run(["g++", "-std=c++17", "-Wall", "-Werror", "-fsyntax-only", "-x", "c++", hdr], check=True)
