"""CPU-side checks of the C ABI: the library builds, loads, exports every declared symbol, and
rejects bad arguments on the host before touching a GPU.  No compute call is made here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def M():
    from paper_2511_06010_b200 import build

    build.build()
    from paper_2511_06010_b200 import binding

    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "moska.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moska_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(M):
    names = declared_symbols()
    assert len(names) >= 12
    lib = ctypes.CDLL(M.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in moska.h but not exported"
        assert n in M.EXPORTS, f"{n} has no Python binding"
        assert hasattr(M, n[len("moska_"):]), f"binding function for {n} missing"
    assert M.version() >= 100


def test_header_is_plain_c_and_a_c_program_links_against_the_library(M, tmp_path):
    """include/moska.h compiles as C99 with warnings as errors, and a C program that includes it
    links against the shared library and runs its host-only calls (no GPU needed)."""
    import shutil
    import subprocess

    gcc = shutil.which("gcc")
    if gcc is None:
        pytest.skip("no C compiler")
    src = tmp_path / "use_moska.c"
    src.write_text(
        '#include <stdio.h>\n#include "moska.h"\n'
        "int main(void) {\n"
        "    moska_shape s = {64, 32, 8, 128, 128, 512, 8, 8, 4, 0, 0};\n"
        "    if (moska_version() < 100) return 1;\n"
        "    if (moska_partial_slots(&s) != 12) return 2;\n"
        "    if (moska_workspace_bytes(&s) == 0) return 3;\n"
        "    s.k = 1000; /* k > C */\n"
        "    if (moska_workspace_bytes(&s) != 0) return 4;\n"
        '    printf("%s\\n", moska_last_error());\n'
        "    return 0;\n}\n")
    exe = tmp_path / "use_moska"
    lib_dir = os.path.dirname(M.LIB_PATH)
    subprocess.run([gcc, "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(ROOT, "include"),
                    str(src), "-o", str(exe), "-L", lib_dir, "-l:" + os.path.basename(M.LIB_PATH),
                    "-Wl,-rpath," + lib_dir], check=True, capture_output=True, text=True)
    r = subprocess.run([str(exe)], capture_output=True, text=True, timeout=60)
    assert r.returncode == 0, (r.returncode, r.stdout, r.stderr)
    assert r.stdout.strip() != ""   # the text of the rejected shape


def test_pure_host_helpers(M):
    s = M.shape(64, 32, 8, 128, 128, 512, 8, n_unique_splits=4)
    assert M.partial_slots(s) == 12
    assert M.workspace_bytes(s) > 256 and M.workspace_bytes(s) % 256 == 0
    assert 1 <= M.default_unique_splits(64, 8, 4096) <= 8
    assert M.default_unique_splits(1024, 8, 32768) >= 1
    assert M.default_unique_splits(4, 1, 100) == 1
    # the FP8 kernel has shorter-lived CTAs: never fewer splits than one, capped by the context
    assert M.default_unique_splits_fp8(64, 8, 4096) == 4
    assert M.default_unique_splits_fp8(4, 1, 100) == 1
    assert 1 <= M.default_unique_splits_fp8(1, 8, 1 << 20) <= 64


@pytest.mark.parametrize("kwargs,status", [
    (dict(Hq=30), -1),            # Hq % Hkv != 0
    (dict(D=96), -2),             # unsupported head dim
    (dict(Hq=128), -2),           # G = 16 > 8
    (dict(L=100), -2),            # L not a multiple of 128
    (dict(k=0), -1),
    (dict(k=129), -1),            # k > C
    (dict(q_len=3), -1),          # q_len does not divide B
    (dict(q_len=-1), -1),
])
def test_bad_shapes_are_rejected_on_the_host(M, kwargs, status):
    base = dict(B=4, Hq=32, Hkv=8, D=128, C=128, L=512, k=8)
    base.update(kwargs)
    s = M.shape(**base)
    with pytest.raises(M.MoskaError) as e:
        M.route(0x1000, 0x1000, 0x1000, None, s, stream=0)
    assert e.value.status == status
    assert M.last_error() != ""


def test_null_pointer_and_workspace_errors_come_before_any_launch(M):
    s = M.shape(4, 32, 8, 128, 128, 512, 8)
    with pytest.raises(M.MoskaError) as e:
        M.merge(None, 0x1000, 0x1000, None, None, s, stream=0)
    # NULL is reported as invalid argument unless the device check (no GPU here) comes first
    assert e.value.status in (M.ERR_INVALID_ARG, M.ERR_CUDA, M.ERR_UNSUPPORTED)
    # several query tokens per request: more than 16 rows per (request, KV head), D = 64 and the
    # FP8 store are refused before anything is launched
    for kw, call in ((dict(Hq=64, q_len=4), "bf16"), (dict(D=64, q_len=2), "bf16"), (dict(q_len=4), "fp8")):
        base = dict(B=4, Hq=32, Hkv=8, D=128, C=128, L=512, k=8)
        base.update(kw)
        sq = M.shape(**base)
        with pytest.raises(M.MoskaError) as e:
            if call == "bf16":
                M.unique_attn(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 1.0, sq, stream=0)
            else:
                M.unique_attn_fp8(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 0x1000,
                                  1.0, sq, stream=0)
        assert e.value.status == M.ERR_UNSUPPORTED
    bad = M.shape(4, 32, 8, 128, 128, 512, 8, shared_slots=0)
    with pytest.raises(M.MoskaError) as e:
        M.partial_slots(bad)
    assert e.value.status == M.ERR_INVALID_ARG
    assert M.workspace_bytes(bad) == 0


def test_misaligned_pointers_are_rejected_on_the_host(M):
    """Every entry point names its alignment (16 bytes for q and the private store, 128 for the
    TMA-read shared store, 32 for the partial outputs, 256 for the workspace); a pointer that
    breaks it is an invalid argument before any launch, whatever the other arguments are."""
    s = M.shape(4, 32, 8, 128, 128, 512, 8)
    A = 0x10000  # aligned to everything asked for
    cases = [
        lambda: M.route(A + 2, A, A, None, s, stream=0),
        lambda: M.route(A, A + 4, A, None, s, stream=0),
        lambda: M.build_chunk_summaries(A + 8, A, s, stream=0),
        lambda: M.shared_attn(A, A + 64, A, A, A, A, A, A, 1.0, s, None, stream=0),
        lambda: M.shared_attn(A, A, A + 16, A, A, A, A, A, 1.0, s, None, stream=0),
        lambda: M.shared_attn(A, A, A, A, A, A, A + 16, A, 1.0, s, None, stream=0),
        lambda: M.unique_attn(A, A + 2, A, A, A, A, A, 1.0, s, stream=0),
        lambda: M.unique_attn(A, A, A, A + 4, A, A, A, 1.0, s, stream=0),
        lambda: M.merge(A + 8, A, A, None, None, s, stream=0),
        lambda: M.merge(A, A, A + 2, None, None, s, stream=0),
        lambda: M.gemv_baseline(A, A, A + 8, A, A, A, 1.0, s, stream=0),
        lambda: M.group_by_chunk_noalloc(A + 2, A, A, s, stream=0),
    ]
    for i, call in enumerate(cases):
        with pytest.raises(M.MoskaError) as e:
            call()
        assert e.value.status == M.ERR_INVALID_ARG, f"case {i}: {M.last_error()}"
        assert "aligned" in M.last_error(), f"case {i}: {M.last_error()}"
    # a misaligned (or missing) workspace is a workspace error
    import ctypes

    lib = ctypes.CDLL(M.LIB_PATH)
    lib.moska_group_by_chunk.restype = ctypes.c_int
    lib.moska_group_by_chunk.argtypes = M.EXPORTS["moska_group_by_chunk"][1]
    need = M.workspace_bytes(s)
    assert lib.moska_group_by_chunk(A, A, A, ctypes.byref(s), A + 128, need, 0) == M.ERR_WORKSPACE
    assert lib.moska_group_by_chunk(A, A, A, ctypes.byref(s), A, need - 1, 0) == M.ERR_WORKSPACE


def test_fp8_shared_store_entry_points_reject_bad_arguments_on_the_host(M):
    """The FP8 shared-store calls: D = 64 is refused, misaligned code pointers and a missing
    workspace (needed in dense mode too, for the f16 copy of the queries) are reported before any
    launch, and the host-buffer step insists on its four buffers."""
    A = 0x10000
    s = M.shape(4, 32, 8, 128, 128, 512, 8)
    ws_fake = type("Ws", (), {"numel": lambda self: 1 << 30, "element_size": lambda self: 1,
                              "is_contiguous": lambda self: True, "data_ptr": lambda self: A})()
    with pytest.raises(M.MoskaError) as e:
        M.shared_attn_fp8(A, A, A, A, A, A, A, A, A, A, 1.0, M.shape(4, 32, 8, 64, 128, 512, 8), ws_fake, stream=0)
    assert e.value.status == M.ERR_UNSUPPORTED
    with pytest.raises(M.MoskaError) as e:
        M.shared_attn_fp8(A, A + 64, A, A, A, A, A, A, A, A, 1.0, s, ws_fake, stream=0)
    assert e.value.status == M.ERR_INVALID_ARG and "aligned" in M.last_error()
    # dense mode (no routing arrays) still needs the workspace
    sd = M.shape(4, 32, 8, 128, 128, 512, 128, shared_slots=16)
    with pytest.raises(M.MoskaError) as e:
        M.shared_attn_fp8(A, A, A, A, A, None, None, None, A, A, 1.0, sd, None, stream=0)
    assert e.value.status == M.ERR_WORKSPACE
    # dense mode with more partial slots than chunks
    with pytest.raises(M.MoskaError) as e:
        M.shared_attn_fp8(A, A, A, A, A, None, None, None, A, A, 1.0,
                          M.shape(4, 32, 8, 128, 8, 512, 8, shared_slots=16), ws_fake, stream=0)
    assert e.value.status == M.ERR_INVALID_ARG
    with pytest.raises(M.MoskaError) as e:
        M.decode_step_fp8_host(None, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, 1.0, s, ws_fake, stream=0)
    assert e.value.status == M.ERR_INVALID_ARG
    with pytest.raises(M.MoskaError) as e:
        M.decode_step_fp8_host(A + 2, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, A, 1.0, s, ws_fake, stream=0)
    assert e.value.status == M.ERR_INVALID_ARG
