"""Host-only checks of the C ABI: the library loads without a GPU, exports every declared symbol,
and rejects host-checkable mistakes before any launch."""
import ctypes
import os
import re

import pytest

import __graft_entry__  # noqa: F401  (builds librpx.so on import of build())
from paper_2608_14498_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2608_14498_b200 import build

    build.build()
    return B.load_library()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "rpx.h")).read()
    declared = re.findall(r"RPX_API[^;(]*?\b(rpx_\w+)\s*\(", header)
    assert sorted(declared) == sorted(B.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert B.version() == 100
    seen = set()
    for code in range(0, -10, -1):
        s = B.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 10
    assert B.status_string(-99) == "unknown status"


def test_sm_budget_is_host_state_with_validation(lib):
    assert B.get_sm_budget() == 0
    B.set_sm_budget(96)
    assert B.get_sm_budget() == 96
    with pytest.raises(B.RpxError) as e:
        B.set_sm_budget(-1)
    assert e.value.status == -2 and B.get_sm_budget() == 96  # rejected, unchanged
    B.set_sm_budget(0)
    assert B.get_sm_budget() == 0


def test_workspace_arithmetic(lib):
    # every attention call keeps its work-item counter in the first 256 bytes; fp32 calls (CUDA-core path) use nothing
    # of it but ask for the same piece
    assert B.prefix_attn_workspace_bytes(28, 4, 128, B.RPX_BF16, 32768) == 256
    assert B.prefix_attn_workspace_bytes(28, 4, 128, B.RPX_BF16, 0) == 0
    need = B.prefix_attn_workspace_bytes(4, 2, 64, B.RPX_F32, 256)
    assert need == 256
    # a suffix pass small enough to be split over the cached prefix also gets room for the partials of 4 ranges:
    # arrival counters, (max, sum) pairs and fp32 rows per (token, head)
    split = 512 + 4 * 128 * 8 + 4 * 128 * 64 * 4
    assert B.suffix_attn_workspace_bytes(4, 2, 64, B.RPX_BF16, 32) == 256 + split
    assert B.suffix_attn_workspace_bytes(4, 2, 64, B.RPX_F32, 32) == 256
    assert B.suffix_attn_workspace_bytes(28, 4, 128, B.RPX_BF16, 113377) == 256  # too many rows to be worth splitting
    # 152064 columns = 594 tiles of 256; one float4 per (chunk, row): 38 chunks of 16 tiles up to 191 row
    # tiles of 128 rows, 75 chunks of 8 tiles from 192 row tiles on
    assert B.token_logprobs_workspace_bytes(12800, 3584, 152064, B.RPX_BF16) == 38 * 12800 * 16
    assert B.token_logprobs_workspace_bytes(34816, 3584, 152064, B.RPX_BF16) == 75 * 34816 * 16
    f32 = B.token_logprobs_workspace_bytes(288, 256, 4096, B.RPX_F32)
    # up to 64 row tiles the chunk length (2..8 tiles) is the one with the fewest rounds on 148 SMs:
    # 3 row tiles x 16 vocabulary tiles -> 2-tile chunks, 8 of them
    assert f32 == 8 * 288 * 16 + 288 * 256 * 2 + 4096 * 256 * 2
    # 16 row tiles x 594 vocabulary tiles -> 5-tile chunks, 119 of them (65 tile-times against 64.2 ideal)
    assert B.token_logprobs_workspace_bytes(2048, 3584, 152064, B.RPX_BF16) == 119 * 2048 * 16
    assert B.token_logprobs_workspace_bytes(0, 256, 4096, B.RPX_BF16) == 0


def _attn_call(lib, desc, q=0x1000, k=0x1000, v=0x1000, strides=(512, 256, 256), cu=0x1000, batch=1, total=16,
               max_len=16, cache=None, out=0x1000, ws=None, ws_bytes=0):
    return lib.rpx_prefix_attn(ctypes.byref(desc), q, k, v, strides[0], strides[1], strides[2], cu, batch, total, max_len,
                               cache, out, None, ws, ws_bytes, None, None)


def test_attention_rejects_bad_arguments_before_any_launch(lib):
    good = B.AttnDesc(4, 2, 128, 0.0, B.RPX_BF16)
    assert lib.rpx_prefix_attn(None, 0x1000, 0x1000, 0x1000, 512, 256, 256, 0x1000, 1, 16, 16, None, 0x1000, None, None,
                               0, None, None) == -1
    assert _attn_call(lib, B.AttnDesc(4, 3, 128, 0.0, B.RPX_BF16)) == -2  # heads not divisible
    assert _attn_call(lib, B.AttnDesc(4, 2, 96, 0.0, B.RPX_BF16)) == -2  # head_dim
    assert _attn_call(lib, B.AttnDesc(4, 2, 128, 0.0, 7)) == -3  # dtype
    assert _attn_call(lib, good, q=None) == -1
    assert _attn_call(lib, good, q=0x1008) == -4
    assert _attn_call(lib, good, strides=(516, 256, 256)) == -4
    assert _attn_call(lib, good, strides=(256, 256, 256)) == -2  # token stride shorter than a row
    assert _attn_call(lib, good, total=-1) == -2
    assert _attn_call(lib, B.AttnDesc(4, 2, 128, 0.0, B.RPX_F32), ws=None, ws_bytes=0) == -5
    # a workspace that is large enough but sits on a 16-byte boundary only (say, cut out of an arena): the kernels'
    # work-item counter and split-KV partials are accessed with up to 32-byte vector instructions
    assert _attn_call(lib, good, ws=0x10010, ws_bytes=1 << 20) == -4
    assert _attn_call(lib, good, ws=0x10080, ws_bytes=1 << 20) == -4
    ok_cache_s = B.KvCache(0x1000, 0x1000, 8, 16, 0x1000, 4)
    assert lib.rpx_suffix_attn(ctypes.byref(good), 0x1000, 0x1000, 0x1000, 512, 256, 256, 0x1000, 0x1000, 1, 16, 16, 64,
                               ctypes.byref(ok_cache_s), 0x1000, None, 0x10010, 1 << 24, None, None) == -4
    # legal no-ops need neither pointers nor a device
    assert _attn_call(lib, good, q=None, batch=0, total=0) == 0
    assert _attn_call(lib, good, q=None, total=0) == 0
    bad_cache = B.KvCache(0x1000, 0x1000, 8, 32, 0x1000, 4)
    assert _attn_call(lib, good, cache=ctypes.byref(bad_cache)) == -2  # block size must be 16
    null_cache = B.KvCache(None, 0x1000, 8, 16, 0x1000, 4)
    assert _attn_call(lib, good, cache=ctypes.byref(null_cache)) == -1
    # the suffix pass needs a cache and prefix lengths
    rc = lib.rpx_suffix_attn(ctypes.byref(good), 0x1000, 0x1000, 0x1000, 512, 256, 256, 0x1000, 0x1000, 1, 16, 16, 64,
                             None, 0x1000, None, None, 0, None, None)
    assert rc == -1
    # and so does chunked prefill
    rc = lib.rpx_chunk_attn(ctypes.byref(good), 0x1000, 0x1000, 0x1000, 512, 256, 256, 0x1000, 0x1000, 1, 16, 16, 64,
                            None, 0x1000, None, None, 0, None, None)
    assert rc == -1
    ok_cache = B.KvCache(0x1000, 0x1000, 8, 16, 0x1000, 4)
    rc = lib.rpx_chunk_attn(ctypes.byref(good), 0x1000, 0x1000, 0x1000, 512, 256, 256, 0x1000, None, 1, 16, 16, 64,
                            ctypes.byref(ok_cache), 0x1000, None, None, 0, None, None)
    assert rc == -1  # cached_lens missing


def test_attention_backward_rejects_bad_arguments_before_any_launch(lib):
    def call(desc=None, q=0x1000, dout=0x1000, lse=0x1000, dq=0x1000, strides=(512, 256, 256), total=16, ws=0x10000,
             ws_bytes=1 << 20, batch=1):
        desc = desc or B.AttnDesc(4, 2, 128, 0.0, B.RPX_BF16)
        return lib.rpx_attn_backward(ctypes.byref(desc), q, 0x1000, 0x1000, strides[0], strides[1], strides[2], 0x1000,
                                     dout, lse, 0x1000, None, None, batch, total, 16, dq, 0x1000, 0x1000, 0, ws, ws_bytes,
                                     None, None)

    assert call(desc=B.AttnDesc(4, 2, 128, 0.0, B.RPX_F32)) == -3   # bf16 only
    assert call(desc=B.AttnDesc(4, 3, 128, 0.0, B.RPX_BF16)) == -2
    assert call(q=None) == -1
    assert call(dout=None) == -1
    assert call(lse=None) == -1
    assert call(dq=0x1008) == -4
    assert call(strides=(256, 256, 256)) == -2
    assert call(ws=None) == -5
    assert call(ws_bytes=16) == -5          # 16 tokens x 4 heads x 4 bytes = 256 are needed
    assert call(ws=0x10010) == -4
    assert call(total=0, q=None) == 0 and call(batch=0, q=None) == 0
    good = B.AttnDesc(28, 4, 128, 0.0, B.RPX_BF16)
    assert lib.rpx_attn_backward_workspace_bytes(ctypes.byref(good), 1000) == 112128  # 1000 x 28 x 4 = 112000 rounded up to 256
    assert lib.rpx_attn_backward_workspace_bytes(ctypes.byref(good), 3) == 512


def test_logprobs_rejects_bad_arguments_before_any_launch(lib):
    def call(hidden=0x1000, stride=256, w=0x1000, ids=0x1000, n=8, h=256, v=4096, dt=B.RPX_BF16, lp=0x1000, ws=0x1000,
             ws_bytes=1 << 30):
        return lib.rpx_token_logprobs(hidden, stride, w, ids, n, h, v, dt, lp, None, ws, ws_bytes, None, None)

    assert call(dt=5) == -3
    assert call(h=100) == -2
    assert call(v=0) == -2
    assert call(hidden=None) == -1
    assert call(lp=None) == -1
    assert call(stride=128) == -2
    assert call(stride=260) == -4
    assert call(w=0x1004) == -4
    assert call(ws=None) == -5
    assert call(ws_bytes=16) == -5
    assert call(ws=0x1010) == -4  # workspaces are 256-byte aligned
    assert call(n=0, hidden=None) == 0


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "_LIB_PATH", str(tmp_path / "librpx.so"))
    with pytest.raises(FileNotFoundError):
        B.load_library()
