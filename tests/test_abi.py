"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and its host-only entry points behave."""
import re
import subprocess
from pathlib import Path

import pytest

import paper_2602_19128_b200 as moe
from paper_2602_19128_b200 import binding
from paper_2602_19128_b200.build import build_library

ROOT = Path(__file__).resolve().parent.parent


def declared_symbols():
    text = (ROOT / "include" / "moe.h").read_text() + (ROOT / "include" / "gqa_decode.h").read_text()
    return sorted(set(re.findall(r"MOE_API[^;(]*?\b((?:moe|gqa)_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build_library()
    L = moe.lib()
    names = declared_symbols()
    assert len(names) >= 10
    assert sorted(names) == sorted(binding.EXPORTED)
    for n in names:
        assert hasattr(L, n), n


@pytest.mark.parametrize("compiler,std,suffix", [("gcc", "-std=c99", ".c"), ("g++", "-std=c++11", ".cpp")])
def test_header_stands_alone_in_c_and_cxx(tmp_path, compiler, std, suffix):
    """The boundary is a C ABI: the header must compile by itself, as strict C and as C++, with no CUDA or
    torch header on the include path, and a caller must be able to take the address of every entry point."""
    src = tmp_path / ("use_header" + suffix)
    body = "".join(f"    p[{i}] = (const void *)&{n};\n" for i, n in enumerate(declared_symbols()))
    src.write_text('#include "moe.h"\n#include "gqa_decode.h"\n#include "moe.h"\n#include "gqa_decode.h"\n'  # twice: the include guards hold
                   f"const void *p[{len(declared_symbols())}];\n"
                   "void take_addresses(void) {\n" + body + "}\n")
    r = subprocess.run([compiler, std, "-Wall", "-Wextra", "-Werror", "-I", str(ROOT / "include"),
                        "-c", str(src), "-o", str(tmp_path / "use_header.o")], capture_output=True, text=True)
    assert r.returncode == 0, r.stderr


def test_workspace_size_and_layout_are_consistent():
    for cfg in [(16, 256, 512, 8, 2), (512, 4096, 14336, 8, 2), (128, 7168, 2048, 256, 8),
                (8192, 7168, 2048, 256, 8), (4096, 4096, 1536, 128, 8)]:
        n = moe.moe_workspace_bytes(*cfg)
        L = moe.moe_workspace_layout(*cfg)
        assert n == L.total_bytes > 0
        offs = [L.status, L.topk_ids, L.topk_weights, L.expert_offsets, L.sorted_to_flat, L.flat_to_sorted,
                L.route_scratch, L.x_perm, L.h, L.y, L.staging]
        assert offs == sorted(offs) and all(o % 256 == 0 for o in offs) and offs[-1] < n
        T, H, I, E, k = cfg
        assert L.h - L.x_perm >= T * k * H * 2 and L.y - L.h >= T * k * I * 2
    # outside the envelope: size 0
    assert moe.moe_workspace_bytes(16, 200, 512, 8, 2) == 0      # H not a multiple of 128
    assert moe.moe_workspace_bytes(16, 256, 512, 300, 2) == 0    # E > 256
    assert moe.moe_workspace_bytes(16, 256, 512, 8, 9) == 0      # top_k > E
    assert moe.moe_route_workspace_bytes(128, 256, 8) > 0
    assert moe.moe_route_workspace_bytes(128, 0, 1) == 0


def test_status_strings_and_launch_count():
    assert moe.moe_status_string(0) == "ok"
    assert "wait" in moe.moe_status_string(-7)
    assert moe.moe_status_string(-99) == "unknown status"
    assert moe.moe_forward_launch_count(0) == 0 and moe.moe_forward_launch_count(16) == 5
    assert moe.moe_forward_launch_count(1024) == 5 and moe.moe_forward_launch_count(1025) == 7


def test_token_tile_bound_follows_the_mean_rows_per_expert():
    assert moe.moe_token_tile_rows(16, 256, 512, 8, 2) == 32            # 4 rows per expert
    assert moe.moe_token_tile_rows(128, 7168, 2048, 256, 8) == 32
    assert moe.moe_token_tile_rows(512, 4096, 14336, 8, 2) == 256       # 128 rows per expert: experts fit 256
    assert moe.moe_token_tile_rows(8192, 7168, 2048, 256, 8) == 320     # 256 on average: one wide tile per expert
    assert moe.moe_token_tile_rows(4096, 4096, 1536, 128, 8) == 320
    assert moe.moe_token_tile_rows(8192, 7168, 2048, 208, 8) == 384     # 315 on average
    assert moe.moe_token_tile_rows(8192, 7168, 2048, 128, 8) == 256     # 512 on average: several tiles per expert anyway
    assert moe.moe_token_tile_rows(8192, 7168, 2048, 256, 8, binding.MOE_FLAG_NARROW_TILES) == 256
    assert moe.moe_token_tile_rows(8192, 7040, 2048, 256, 8) == 256     # H not a multiple of 256: no wide-tile kernel
    assert moe.moe_token_tile_rows(8192, 7168, 2048, 300, 8) == 0       # outside the envelope


def test_mx_layout():
    for cfg in [(16, 256, 512, 8, 2), (512, 4096, 14336, 8, 2), (128, 7168, 2048, 256, 8), (8192, 7168, 2048, 256, 8)]:
        n = moe.moe_mxfp8_workspace_bytes(*cfg)
        L = moe.moe_mxfp8_workspace_layout(*cfg)
        T, H, I, E, k = cfg
        A = T * k
        assert n == L.total_bytes > 0
        offs = [L.status, L.topk_ids, L.topk_weights, L.expert_offsets, L.sorted_to_flat, L.flat_to_sorted,
                L.route_scratch, L.x_q, L.x_sf, L.h_q, L.h_sf, L.y, L.staging]
        assert offs == sorted(offs) and all(o % 256 == 0 for o in offs) and offs[-1] < n
        assert L.tile_rows in (32, 64, 128, 160, 240, 304, 384)
        atoms_per_tile = (L.tile_rows + 127) // 128
        assert L.sf_atoms == (A // min(L.tile_rows, 256) + E + 1) * atoms_per_tile
        assert L.x_sf - L.x_q >= A * H and L.h_q - L.x_sf >= (H // 128) * L.sf_atoms * 512
        assert L.y - L.h_sf >= (I // 128) * L.sf_atoms * 512
    assert moe.moe_mxfp8_workspace_layout(512, 4096, 14336, 8, 2).tile_rows == 160     # 128 rows per expert on average
    assert moe.moe_mxfp8_workspace_layout(8192, 7168, 2048, 256, 8).tile_rows == 304   # 256 on average: one wide tile per expert
    assert moe.moe_mxfp8_workspace_layout(8192, 7168, 2048, 208, 8).tile_rows == 384   # 315 on average
    assert moe.moe_mxfp8_workspace_layout(8192, 7168, 2048, 128, 8).tile_rows == 240   # 512 on average: several tiles anyway
    assert moe.moe_mxfp8_workspace_layout(8192, 7040, 2048, 256, 8).tile_rows == 128   # H not a multiple of 256
    assert moe.moe_mxfp8_workspace_bytes(16, 256, 192, 8, 2) == 0                      # I must be a multiple of 128


def test_argument_errors_are_reported_before_any_launch():
    """Host-side validation needs no GPU: nothing is launched for an empty batch or a rejected argument."""
    L = moe.lib()
    null = None
    assert L.moe_forward(null, null, null, null, 0, 256, 512, 8, 2, null, null, 0, null) == 0          # T == 0
    assert L.moe_forward(null, null, null, null, -1, 256, 512, 8, 2, null, null, 0, null) == -2        # shape
    assert L.moe_forward(null, null, null, null, 4, 200, 512, 8, 2, null, null, 0, null) == -3         # envelope
    assert L.moe_forward(null, null, null, null, 4, 256, 512, 8, 2, null, null, 0, null) == -1         # NULL
    assert L.moe_forward_mxfp8(null, null, null, null, null, null, 0, 256, 128, 8, 2, null, 0, 8, null, null, 0, null, null) == 0
    assert L.moe_forward_mxfp8(null, null, null, null, null, null, 4, 256, 192, 8, 2, null, 0, 8, null, null, 0, null, null) == -3
    assert L.moe_forward_mxfp8(null, null, null, null, null, null, 4, 256, 128, 8, 2, null, 6, 4, null, null, 0, null, null) == -2
    router = binding.grouped_router(3, 1)   # 8 experts do not split into 3 groups
    import ctypes
    assert L.moe_forward_grouped(null, null, null, null, 4, 256, 512, 8, 2, ctypes.byref(router), 0, 8, null, null, 0, null, 0) == -3
    assert L.moe_forward_grouped(null, null, null, null, 4, 256, 512, 8, 2, None, 0, 8, null, null, 0, null, 0) == -1
    router = binding.grouped_router(4, 1)   # one eligible group of two experts cannot supply top_k = 3
    assert L.moe_route_grouped(null, 4, 8, 3, ctypes.byref(router), null, null, null, null, null, null, 0, null) == -3


def test_router_entry_points_share_one_argument_check():
    """moe_route, moe_route_grouped and moe_route_static validate their arrays the same way, on the host, before
    anything touches the device: a NULL array is -1, an array that is not 4-byte aligned is -4 (fake addresses are
    enough: a rejected call never dereferences them), and the static variant reports its size limit first."""
    import ctypes
    L = moe.lib()
    ok, odd = 0x10000, 0x10002
    router = binding.grouped_router(1, 1)
    for bad_slot in range(6):   # logits, ids, weights, offsets, sorted_to_flat, flat_to_sorted
        arrays = [odd if i == bad_slot else ok for i in range(6)]
        assert L.moe_route(arrays[0], 4, 8, 2, *arrays[1:], ok, 1 << 20, None) == -4
        assert L.moe_route_static(arrays[0], 4, 8, 2, *arrays[1:], None) == -4
        assert L.moe_route_grouped(arrays[0], 4, 8, 2, ctypes.byref(router), *arrays[1:], ok, 1 << 20, None) == -4
        arrays = [None if i == bad_slot else ok for i in range(6)]
        assert L.moe_route(arrays[0], 4, 8, 2, *arrays[1:], ok, 1 << 20, None) == -1
        assert L.moe_route_static(arrays[0], 4, 8, 2, *arrays[1:], None) == -1
    assert L.moe_route_static(ok, 4, 8, 9, ok, ok, ok, ok, ok, None) == -2            # top_k > E
    assert L.moe_route_static(ok, 4, 300, 2, ok, ok, ok, ok, ok, None) == -3           # E > 256
    assert L.moe_route_static(odd, 16288, 256, 8, odd, ok, ok, ok, ok, None) == -9     # the size limit comes first
    assert L.moe_route(ok, 4, 8, 2, ok, ok, ok, ok, ok, ok + 64, 1 << 20, None) == -4  # workspace: 256-byte aligned
    assert L.moe_route(ok, 4, 8, 2, ok, ok, ok, ok, ok, ok, 16, None) == -5            # workspace too small
    assert "2^27" in moe.moe_status_string(-3)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    """No fallback: with the shared library absent, the binding raises instead of computing anything elsewhere."""
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", tmp_path / "libmoe_b200.so")
    with pytest.raises(FileNotFoundError, match="no fallback"):
        moe.moe_workspace_bytes(16, 256, 512, 8, 2)


def test_product_sources_never_reach_the_oracle():
    """The oracle is test infrastructure: nothing in the package (Python or CUDA) imports, includes or names it."""
    pkg = ROOT / "paper_2602_19128_b200"
    for f in sorted(pkg.rglob("*")):
        if f.suffix in (".py", ".cu", ".cuh", ".h"):
            text = f.read_text()
            assert not re.search(r"^\s*(from|import)\s+oracle\b", text, re.M), f
            assert "moe_oracle" not in text and "oracle/" not in text, f
    for f in sorted((ROOT / "oracle").rglob("*")):  # and the oracle reaches nothing of the product but the input recipe
        if f.suffix in (".py", ".c", ".h"):
            text = f.read_text()
            assert "csrc" not in text and "binding" not in text and "libmoe_b200" not in text, f
