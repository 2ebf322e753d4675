"""Host-side checks that need no GPU: the shared library loads, exports every function the
header declares, reports workspace sizes, and rejects bad arguments before touching CUDA."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_40335_b200 import binding, build
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "dp_ghost.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2609_40335_b200 import binding
    names = _declared_functions()
    assert {"dp_ghost_norms", "dp_embed_norms", "dp_tied_cross_term", "dp_clip_accumulate",
            "dp_add_noise"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(binding.EXPORTS)
    assert b"sm_100a" in lib.dp_version()


def test_bad_arguments_return_status_without_cuda(lib):
    from paper_2609_40335_b200.binding import _LinearDesc
    assert lib.dp_ghost_norms(None, 1, 1, 2, 16, None, None, 0, None, None) == 1
    d = (_LinearDesc * 1)()
    assert lib.dp_ghost_norms(d, 1, 1, 2, 16, C.c_void_p(256), None, 0, None, None) == 1   # null A / G
    d[0].A, d[0].G, d[0].d, d[0].p, d[0].lda, d[0].ldg = 4096, 8192, 64, 64, 64, 64
    d[0].mode = 9
    assert lib.dp_ghost_norms(d, 1, 1, 2, 16, C.c_void_p(256), None, 0, None, None) == 1   # bad mode
    d[0].mode = 0
    d[0].A = 4098
    assert lib.dp_ghost_norms(d, 1, 1, 2, 16, C.c_void_p(256), None, 0, None, None) == 3   # alignment
    d[0].A = 4096
    d[0].lda = 68
    assert lib.dp_ghost_norms(d, 1, 1, 2, 16, C.c_void_p(256), None, 0, None, None) == 3   # ld % 8
    d[0].lda = 64
    assert lib.dp_ghost_norms(d, 1, 1, 2, 16, C.c_void_p(256), None, 0, None, None) == 4   # no workspace
    assert lib.dp_clip_factors(C.c_void_p(256), 4, C.c_float(0.0), C.c_void_p(512), None, None) == 1
    assert lib.dp_add_noise(C.c_void_p(256), 8, C.c_float(-1.0), C.c_float(1.0), C.c_float(1.0), 0, 0, 0, None) == 1
    assert lib.dp_add_noise(C.c_void_p(260), 8, C.c_float(1.0), C.c_float(1.0), C.c_float(1.0), 0, 0, 0, None) == 3
    assert lib.dp_embed_norms(C.c_void_p(256), C.c_void_p(512), 64, 1, 2, 5000, 64, 100, C.c_void_p(768),
                              None, C.c_void_p(1024), 1 << 20, None, None) == 2              # T too large
    assert lib.dp_status_string(3).decode().startswith("pointer")


def test_workspace_sizes_follow_the_plan(lib):
    from paper_2609_40335_b200.binding import _LinearDesc
    d = (_LinearDesc * 2)()
    for k, (dd, pp) in enumerate([(768, 2304), (768, 50257)]):
        d[k].A, d[k].G, d[k].d, d[k].p, d[k].lda, d[k].ldg, d[k].mode = 4096, 8192, dd, pp, dd, (pp + 7) // 8 * 8, 1
    B, T = 32, 128
    n = lib.dp_ghost_norms_ws_bytes(d, 2, 1, B, T)
    # one partial per (example, layer, column chunk): the head is split into several chunks
    assert n >= B * (1 + 8) * 4 and n % 256 == 0
    # fp32 layers of this size run on the tensor cores with their operands split into two bf16
    # terms: the widened operands of the LARGEST layer (two sides, three column blocks, 2 bytes)
    # plus its partial sums; layers too small for a tensor-core tile need nothing
    f32 = lib.dp_ghost_norms_ws_bytes(d, 2, 0, B, T)
    widened = 2 * 3 * B * T * (768 + 50264) * 2
    assert widened <= f32 <= widened + (1 << 20) and f32 % 256 == 0
    tiny = (_LinearDesc * 1)()
    tiny[0].A, tiny[0].G, tiny[0].d, tiny[0].p, tiny[0].lda, tiny[0].ldg, tiny[0].mode = 4096, 8192, 64, 64, 64, 64, 0
    assert lib.dp_ghost_norms_ws_bytes(tiny, 1, 0, 4, 16) == 0
    # few output tiles -> K is split and partial planes are needed; many tiles -> the clip factors
    # and, for a layer as lopsided as the LM head, the pre-scaled bf16 copy of its narrow operand
    small = lib.dp_clip_accumulate_ws_bytes(1, B, T, 768, 768)
    big = lib.dp_clip_accumulate_ws_bytes(1, B, T, 768, 50257)
    mid = lib.dp_clip_accumulate_ws_bytes(1, 64, 256, 3072, 4096)      # many tiles, balanced widths
    assert small > 768 * 768 * 4 and big == 256 + B * T * 768 * 2 and mid == 256
    assert lib.dp_clip_accumulate_embed_ws_bytes(B, T, 768, 50257) >= (4 * 50257 + 50258 + B * T) * 4
