"""CPU-only checks of the boundary: the library builds, loads, and exports what the header declares."""
from __future__ import annotations

import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "castling_attn.h")


def _declared():
    text = open(HEADER).read()
    return sorted(set(re.findall(r"CASTLING_API\s+[\w\s\*]+?\b(castling_attn_\w+)\s*\(", text)))


def test_header_declares_the_entry_points():
    names = _declared()
    for must in ("castling_attn_create", "castling_attn_forward", "castling_attn_destroy",
                 "castling_attn_forward_host"):
        assert must in names


def test_library_exports_every_declared_symbol():
    from paper_2211_10526_b200 import build
    lib = ctypes.CDLL(build.build())
    for name in _declared():
        assert hasattr(lib, name), f"{name} is declared in the header but not exported"


def test_binding_mirrors_the_header():
    from paper_2211_10526_b200 import binding
    for name in _declared():
        assert hasattr(binding, name) or hasattr(binding.lib, name)
    for name in ("castling_attn_create", "castling_attn_forward", "castling_attn_forward_host",
                 "castling_attn_destroy"):
        assert callable(getattr(binding, name))


def test_error_strings_and_workspace_query_need_no_gpu():
    from paper_2211_10526_b200 import binding as b
    codes = [b.OK, b.ERR_INVALID_ARG, b.ERR_UNSUPPORTED, b.ERR_ALIGNMENT, b.ERR_ARCH, b.ERR_CUDA, b.ERR_OOM,
             b.ERR_DEVICE]
    texts = [b.error_string(c) for c in codes]
    assert len(set(texts)) == len(codes) and all(texts)
    assert "unknown" in b.error_string(-99)
    # state + no partials for a small grid: header + BH * (d*d + 2d) floats (S, s and room for the key-row sum
    # of the row-normalised variant)
    assert b.castling_attn_workspace_bytes(2, 4, 14, 14, 32, b.CASTLING_F32) == 4 * (64 + 8 * (32 * 32 + 2 * 32))
    # bf16 with d = 32 may run the tensor-core kernels, which keep 64-wide states
    assert b.castling_attn_workspace_bytes(2, 4, 14, 14, 32, b.CASTLING_BF16) >= 4 * (64 + 8 * (64 * 64 + 64))
    big = b.castling_attn_workspace_bytes(2, 8, 256, 256, 64, b.CASTLING_BF16)
    assert big > 4 * (64 + 16 * (64 * 64 + 64))  # token range is split: partial states too
    assert b.castling_attn_workspace_bytes(0, 4, 14, 14, 32, 0) == 0
    assert b.castling_attn_workspace_bytes(2, 4, 14, 14, 33, 0) == 0
    assert b.castling_attn_workspace_bytes(2, 4, 14, 14, 32, 7) == 0


def test_create_argument_validation_precedes_device_queries():
    """Bad configurations are rejected before any CUDA call, so this runs without a GPU."""
    from paper_2211_10526_b200 import binding as b
    for ksize, code in ((4, b.ERR_INVALID_ARG), (0, b.ERR_INVALID_ARG), (-3, b.ERR_INVALID_ARG), (9, b.ERR_UNSUPPORTED)):
        cfg = b.castling_attn_config_t(ksize, 0.0, 0, 0)
        h = ctypes.c_void_p(123)
        assert b.lib.castling_attn_create(ctypes.byref(cfg), ctypes.byref(h)) == code
        assert h.value is None
    cfg = b.castling_attn_config_t(3, 0.0, 9, 0)
    h = ctypes.c_void_p()
    assert b.lib.castling_attn_create(ctypes.byref(cfg), ctypes.byref(h)) == b.ERR_INVALID_ARG
    assert b.lib.castling_attn_create(ctypes.byref(cfg), None) == b.ERR_INVALID_ARG
    assert b.castling_attn_destroy(None) == b.OK
    assert b.castling_attn_forward(None, 16, 16, 16, 16, None, 16, 1, 1, 1, 1, 32, 0) == b.ERR_INVALID_ARG


def test_workloads_match_the_configured_shapes():
    import workloads
    wl = workloads.WORKLOADS
    assert [c.N for c in wl["c5_sweep_bf16"].calls] == [1024, 4096, 16384, 65536]
    c3 = wl["c3_deit_base_bf16"].calls[0]
    assert (c3.B, c3.H, c3.N, c3.d, c3.ksize, c3.dtype) == (64, 12, 196, 64, 3, "bf16")
    assert c3.algorithmic_bytes == 4 * 64 * 12 * 196 * 64 * 2 + 12 * 64 * 10 * 2
    a = list(workloads.iter_workload("c2_levit_bf16", only=[1]))[0]
    b = list(workloads.iter_workload("c2_levit_bf16"))[1]
    import torch
    assert torch.equal(a.q, b.q) and torch.equal(a.dw_weight, b.dw_weight)
    assert a.q.dtype == torch.bfloat16 and tuple(a.q.shape) == (64, 8, 49, 32)


def test_binding_structs_match_the_header_layout(tmp_path):
    """The ctypes mirrors of the two structs in the header have the C compiler's sizes and field offsets."""
    import subprocess
    from paper_2211_10526_b200 import binding as b
    src = tmp_path / "layout.c"
    src.write_text(
        '#include <stdio.h>\n#include <stddef.h>\n#include "castling_attn.h"\n'
        'int main(void) {\n'
        '  printf("%zu %zu %zu %zu %zu %zu %zu %zu %zu %zu\\n", sizeof(castling_attn_config_t), offsetof(castling_attn_config_t, ksize),\n'
        '         offsetof(castling_attn_config_t, eps), offsetof(castling_attn_config_t, force_path),\n'
        '         offsetof(castling_attn_config_t, max_workspace), offsetof(castling_attn_config_t, prefix_tokens),\n'
        '         offsetof(castling_attn_config_t, normalize_rows), offsetof(castling_attn_config_t, exact_kernel),\n'
        '         offsetof(castling_attn_config_t, sparse_branch), offsetof(castling_attn_config_t, sparse_eps));\n'
        '  printf("%zu %zu %zu %zu\\n", sizeof(castling_attn_layout_t), offsetof(castling_attn_layout_t, q_batch),\n'
        '         offsetof(castling_attn_layout_t, v_head), offsetof(castling_attn_layout_t, out_token));\n'
        '  printf("%d %d %d %u\\n", CASTLING_ERR_SCRATCH_LIMIT, CASTLING_PATH_TENSOR, CASTLING_BF16, CASTLING_STATIC_SCRATCH_BYTES);\n'
        '  return 0;\n}\n')
    exe = tmp_path / "layout"
    subprocess.run(["gcc", "-std=c11", "-I", os.path.join(ROOT, "include"), "-o", str(exe), str(src)], check=True)
    lines = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split("\n")
    cfg, lay = b.castling_attn_config_t, b.castling_attn_layout_t
    assert [int(x) for x in lines[0].split()] == [ctypes.sizeof(cfg), cfg.ksize.offset, cfg.eps.offset, cfg.force_path.offset,
                                                 cfg.max_workspace.offset, cfg.prefix_tokens.offset,
                                                 cfg.normalize_rows.offset, cfg.exact_kernel.offset, cfg.sparse_branch.offset,
                                                 cfg.sparse_eps.offset]
    assert [int(x) for x in lines[1].split()] == [ctypes.sizeof(lay), lay.q_batch.offset, lay.v_head.offset, lay.out_token.offset]
    assert [int(x) for x in lines[2].split()] == [b.ERR_SCRATCH_LIMIT, b.PATH_TENSOR, b.CASTLING_BF16, b.STATIC_SCRATCH_BYTES]
