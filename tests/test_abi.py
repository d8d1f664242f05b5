"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and its host-only entry points behave."""
import re
from pathlib import Path

import paper_2602_19128_b200 as moe
from paper_2602_19128_b200 import binding
from paper_2602_19128_b200.build import build_library

ROOT = Path(__file__).resolve().parent.parent


def declared_symbols():
    text = (ROOT / "include" / "moe.h").read_text()
    return sorted(set(re.findall(r"MOE_API[^;(]*?\b(moe_[a-z0-9_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    build_library()
    L = moe.lib()
    names = declared_symbols()
    assert len(names) >= 10
    assert sorted(names) == sorted(binding.EXPORTED)
    for n in names:
        assert hasattr(L, n), n


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
