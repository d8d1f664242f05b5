"""Host-side logic of the paged decode-attention entry points (include/gqa_decode.h): the envelope, the choice of
sequence splits and the workspace size.  No GPU: only the pure host functions are called, plus the argument checks
of gqa_paged_decode that come before any CUDA call."""
import ctypes

import pytest

import paper_2602_19128_b200 as moe

# status codes of moe_status_t (include/moe.h)
OK, ERR_NULL, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGN, ERR_WORKSPACE = 0, -1, -2, -3, -4, -5

SHAPES = [(1, 64), (1, 65536), (1, 1 << 20), (4, 32768), (8, 8192), (16, 8192), (64, 100), (64, 2048), (64, 8192),
          (64, 16384), (128, 32768), (256, 2048), (256, 8192), (1024, 2048), (4096, 512)]


@pytest.mark.parametrize("B,L", SHAPES)
def test_splits_are_whole_chunks_and_cover_the_longest_sequence(B, L):
    st = moe.gqa_decode_split_tokens(B, 32, 4, 128, L)
    assert st > 0 and st % 64 == 0
    n = -(-max(L, 1) // st)
    assert 1 <= n <= 128
    assert n * st >= L
    assert n == 1 or st >= 4 * 64                      # no split shorter than four chunks
    # the workspace holds a status word, a counter per (item, kv head) and the partial results of n splits
    need = 256 + B * 4 * 4 + B * 4 * n * 8 * (128 + 2) * 4
    ws = moe.gqa_decode_workspace_bytes(B, 32, 4, 128, L)
    assert need <= ws <= need + 4 * 256 + 256


def test_short_batches_are_not_split_and_one_long_sequence_is():
    assert moe.gqa_decode_split_tokens(256, 32, 4, 128, 2048) == 2048     # 1024 blocks already fill the machine
    assert moe.gqa_decode_split_tokens(64, 32, 4, 128, 2048) == 2048
    one = moe.gqa_decode_split_tokens(1, 32, 4, 128, 65536)
    assert 32 <= 65536 // one <= 128                                       # enough blocks for 148 SMs from 4 heads


def test_the_split_does_not_depend_on_the_group_size_but_the_workspace_does():
    assert moe.gqa_decode_split_tokens(8, 32, 4, 128, 8192) == moe.gqa_decode_split_tokens(8, 4, 4, 128, 8192)
    assert moe.gqa_decode_workspace_bytes(8, 32, 4, 128, 8192) > moe.gqa_decode_workspace_bytes(8, 4, 4, 128, 8192)


@pytest.mark.parametrize("B,Hq,Hkv,D,L", [(-1, 32, 4, 128, 10), (2, 32, 4, 64, 10), (2, 30, 4, 128, 10),
                                           (2, 68, 4, 128, 10), (2, 32, 4, 128, -1), (70000, 8, 8, 128, 10)])
def test_outside_the_envelope_the_sizes_are_zero(B, Hq, Hkv, D, L):
    assert moe.gqa_decode_workspace_bytes(B, Hq, Hkv, D, L) == 0
    assert moe.gqa_decode_split_tokens(B, Hq, Hkv, D, L) == 0


def test_argument_checks_come_before_any_cuda_call():
    """Shape, envelope, null and alignment errors are reported on a machine without a GPU, i.e. before the device is
    touched; the pointers are never dereferenced."""
    lib = moe.lib()
    f = lib.gqa_paged_decode
    f.restype = ctypes.c_int
    f.argtypes = [ctypes.c_void_p] * 6 + [ctypes.c_int] * 7 + [ctypes.c_float] + [ctypes.c_void_p] * 3 + [ctypes.c_size_t, ctypes.c_void_p]
    ok = [0x1000] * 6
    tail = (0x2000, None, 0x4000, 1 << 30, None)       # out, lse, workspace, workspace_bytes, stream

    def call(ptrs=ok, B=2, Hq=32, Hkv=4, D=128, P=16, pages=8, L=100, out_ws=tail):
        return f(*ptrs, B, Hq, Hkv, D, P, pages, L, 0.1, *out_ws)
    assert call(P=0) == ERR_SHAPE
    assert call(D=64) == ERR_UNSUPPORTED
    assert call(Hq=30) == ERR_UNSUPPORTED
    assert call(P=1 << 20, pages=1 << 12) == ERR_UNSUPPORTED          # slot numbers would not fit 32 bits
    assert call(B=0) == OK                                           # nothing to do, nothing launched
    assert call(ptrs=[0x1000, None] + [0x1000] * 4) == ERR_NULL
    assert call(ptrs=[0x1008] + [0x1000] * 5) == ERR_ALIGN            # q must be 16-byte aligned
    assert call(ptrs=[0x1000] * 3 + [0x1002] + [0x1000] * 2) == ERR_ALIGN
    assert call(out_ws=(0x2000, None, 0x4010, 1 << 30, None)) == ERR_ALIGN
    assert call(out_ws=(0x2000, None, 0x4000, 16, None)) == ERR_WORKSPACE
