"""CPU-side checks of the C-ABI library: it loads without a GPU, exports every
symbol the public header declares, sizes workspaces on the host and refuses
bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def ngc():
    from paper_2604_18002_b200 import build
    build.build()
    from paper_2604_18002_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "ngc.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ngc_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(ngc):
    syms = declared_symbols()
    assert set(ngc.EXPORTS) <= set(syms) and len(syms) >= 9
    for s in syms:
        assert hasattr(ngc.lib, s), f"{s} declared in ngc.h but not exported"


def test_version_and_strerror(ngc):
    assert ngc.version() >= 100
    assert ngc.lib.ngc_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -99):
        assert len(ngc.lib.ngc_strerror(code)) > 0


def test_struct_layout_matches_header(ngc):
    # 4 pointers, int64, 8 int32
    assert C.sizeof(ngc.CacheDesc) == 4 * 8 + 8 + 8 * 4
    assert ngc.CacheDesc.rows.offset == 32 and ngc.CacheDesc.L.offset == 40 and ngc.CacheDesc.max_len.offset == 64
    assert ngc.CacheDesc.lens_lists.offset == 68


def test_workspace_sizes_on_host(ngc):
    def desc(L, B, Hq, Hkv, d, dtype, rows, max_len):
        return ngc.CacheDesc(1, 1, 1, 1, rows, L, B, Hq, Hkv, d, dtype, max_len)
    big = desc(28, 64, 12, 2, 128, ngc.BF16, 64 * 4096, 4096)
    # sized for the worst layer range (a one-layer call splits along tokens); a few MB at most
    wb = ngc.lib.ngc_workspace_bytes(ngc.OP_DECODE, C.byref(big), 1, 0, 0)
    assert 0 < wb < 8 * 2 ** 20 and wb % 256 == 0
    small = desc(1, 4, 4, 4, 64, ngc.F32, 4 * 512, 512)
    w = ngc.lib.ngc_workspace_bytes(ngc.OP_DECODE, C.byref(small), 1, 0, 0)
    assert w > 0 and w % 256 == 0
    assert ngc.lib.ngc_workspace_bytes(ngc.OP_SAMPLE, C.byref(big), 1, 16384, 8192) == 0
    assert ngc.lib.ngc_workspace_bytes(ngc.OP_SAMPLE, C.byref(big), 1, 16385, 8192) == 64 * 32768 * 8
    assert ngc.lib.ngc_workspace_bytes(ngc.OP_LOGPROB, C.byref(big), 1, 4096, 2048) == 0
    assert ngc.lib.ngc_workspace_bytes(ngc.OP_COMPACT, C.byref(big), 1, 4096, 2048) == 0
    s = ngc.lib.ngc_workspace_bytes(ngc.OP_SCORE, C.byref(big), 1, 4096, 2048)
    assert s >= 28 * 2 * 64 * 4096 * 4


def test_bad_arguments_are_refused_before_launch(ngc):
    lib = ngc.lib
    good = ngc.CacheDesc(1, 1, 1, 1, 16, 1, 1, 2, 1, 64, ngc.F32, 16)
    assert lib.ngc_compact_kv(None, 1, 1, 4, 0, 1, None, None) == -1
    assert lib.ngc_compact_kv(C.byref(good), None, 1, 4, 0, 1, None, None) == -1
    assert lib.ngc_compact_kv(C.byref(good), 1, 1, 4, 3, 1, None, None) == -1
    bad_d = ngc.CacheDesc(1, 1, 1, 1, 16, 1, 1, 2, 1, 48, ngc.F32, 16)
    assert lib.ngc_compact_kv(C.byref(bad_d), 1, 1, 4, 0, 1, None, None) == -1
    bad_g = ngc.CacheDesc(1, 1, 1, 1, 16, 1, 1, 3, 2, 64, ngc.F32, 16)
    assert lib.ngc_decode_attn_ragged(C.byref(bad_g), 1, None, None, 0, 1, 1.0, 1, 0, None, 0, None, None) == -1
    assert lib.ngc_decode_attn_ragged(C.byref(good), 1, None, None, 0, 2, 1.0, 1, 0, None, 0, None, None) == -1
    assert lib.ngc_decode_attn_ragged(C.byref(good), 1, 1, None, 0, 1, 1.0, 1, 0, None, 0, None, None) == -1
    assert lib.ngc_decode_attn_ragged(C.byref(good), 1, None, None, 0, 1, 1.0, 1, ngc.BF16, None, 0, None, None) == -1
    assert lib.ngc_sample_evict(None, 1, None, 1, 1, 1, 8, 4, 0, 0, 0, 0, 1, 1, None, None, 0, None, None) == -1
    assert lib.ngc_sample_evict(1, 1, None, 1, 1, 1, 0, 4, 0, 0, 0, 0, 1, 1, None, None, 0, None, None) == -1
    # a list longer than the shared-memory sorter needs a workspace
    assert lib.ngc_sample_evict(1, 1, None, 1, 1, 1, 20000, 4, 0, 0, 0, 0, 1, 1, None, None, 0, None, None) == -3
    assert lib.ngc_evict_logprob(1, 1, None, 1, None, 1, 1, 1, 8, 4, 1, None, 0, None, None) == -1
    assert lib.ngc_score_evict(C.byref(good), 1, 0, 1, 0, 0, 1, 16, None, None, 0, None, None) == -1
    assert lib.ngc_score_evict(C.byref(good), 1, 5, 1, 0, 0, 1, 8, None, None, 0, None, None) == -1     # n_max too small
    assert lib.ngc_score_evict(C.byref(good), 1, 5, 1, 0, 0, 1, 16, None, None, 0, None, None) == -3    # no workspace
    # a length per layer cannot serve a shared or a per-head eviction list
    per_layer = ngc.CacheDesc(1, 1, 1, 1, 16, 1, 1, 2, 1, 64, ngc.F32, 16, 1)
    assert lib.ngc_compact_kv(C.byref(per_layer), 1, 1, 4, 0, 1, None, None) == -1
    assert lib.ngc_score_evict(C.byref(per_layer), 1, 5, 1, 2, 0, 1, 16, None, None, 0, None, None) == -1
    bad_mode = ngc.CacheDesc(1, 1, 1, 1, 16, 1, 1, 2, 1, 64, ngc.F32, 16, 3)
    assert lib.ngc_compact_kv(C.byref(bad_mode), 1, 1, 4, 0, 1, None, None) == -1


def test_binding_refuses_cpu_tensors(ngc):
    import torch
    t = torch.zeros(4)
    with pytest.raises(ngc.NgcError):
        ngc._ptr(t)


def test_added_entry_points_refuse_bad_arguments(ngc):
    """Gradient, paged and replay entries: null pointers, inconsistent shapes and unsupported layouts are
    turned away on the host (nothing is launched, so this runs without a GPU)."""
    lib = ngc.lib
    bf = ngc.CacheDesc(16, 16, 16, 16, 64, 1, 1, 12, 2, 128, ngc.BF16, 64)      # 16-byte aligned dummy pointers
    f32 = ngc.CacheDesc(16, 16, 16, 16, 16, 1, 1, 2, 1, 64, ngc.F32, 16)
    # log-prob gradient
    assert lib.ngc_evict_logprob_backward(1, 1, None, 1, 1, None, 1, 1, 1, 8, 4, None, None, 0, None, None) == -1   # no output
    assert lib.ngc_evict_logprob_backward(1, 1, None, 1, 1, None, 0, 1, 1, 8, 4, 1, None, 0, None, None) == -1     # no rounds
    # score gradient: fp32 / d = 64 caches are not built; the log variant needs the forward logits; workspace is mandatory
    assert lib.ngc_score_evict_backward(C.byref(f32), 16, 5, 1, 0, 0, None, 16, 16, 16, 16, None, 0, None, None) == -2
    assert lib.ngc_score_evict_backward(C.byref(bf), 16, 5, 1, 0, 1, None, 16, 64, 16, 16, None, 0, None, None) == -1
    assert lib.ngc_score_evict_backward(C.byref(bf), 16, 9, 1, 0, 0, None, 16, 64, 16, 16, None, 0, None, None) == -2  # 6 * 9 rows > 40
    assert lib.ngc_score_evict_backward(C.byref(bf), 16, 5, 1, 0, 0, None, 16, 64, 16, 16, None, 0, None, None) == -3
    # paged cache: page size 32 or 64, bf16 / d = 128 only
    pg = ngc.PagedCacheDesc(16, 16, 16, 16, 1, 1, 12, 2, 128, ngc.BF16, 48, 4, 0)
    assert lib.ngc_decode_attn_paged(C.byref(pg), 16, None, None, 0, 1, 1.0, 16, 0, None, 0, None, None) == -1
    pg = ngc.PagedCacheDesc(16, 16, 16, 16, 1, 1, 4, 4, 64, ngc.F32, 32, 4, 0)
    assert lib.ngc_decode_attn_paged(C.byref(pg), 16, None, None, 0, 1, 1.0, 16, 0, None, 0, None, None) == -2
    assert lib.ngc_score_evict_paged(C.byref(pg), 16, 5, 0, 16, 4, None, None, 0, None, None) == -2
    assert lib.ngc_evict_pages(None, 1, 1, 4, None, None) == -1
    # replay
    assert lib.ngc_replay_visibility(None, 1, 1, 1, 1, 1, 1, 4, 1, 8, 0, 1, 1, None, None) == -1
    assert lib.ngc_replay_visibility(1, 1, 1, 1, 0, 1, 1, 4, 1, 8, 0, 1, 1, None, None) == -1              # no rounds
    assert lib.ngc_replay_visibility(1, 1, 1, 1, 1, 1, 1, 4, 1, 40000, 0, 1, 1, None, None) == -2          # alive set beyond shared memory
    assert lib.ngc_replay_attn(C.byref(f32), 16, 8, None, None, None, 0, 0, 0, 1.0, 16, 0, None, None) == -2
    assert lib.ngc_replay_attn(C.byref(bf), 16, 8, None, None, None, 2, 4, 0, 1.0, 16, 0, None, None) == -1   # rounds without lists
    assert lib.ngc_replay_attn(C.byref(bf), None, 8, None, None, None, 0, 0, 0, 1.0, 16, 0, None, None) == -1
    assert ngc.lib.ngc_workspace_bytes(ngc.OP_SCORE_BACKWARD, C.byref(bf), 1, 0, 0) > 0


def test_bounds_checking_and_nvtx_builds_load_and_export_everything(ngc):
    """The two optional builds (kernels that check their indices; an NVTX range around every call) are separate
    libraries with the same C ABI."""
    from paper_2604_18002_b200 import build
    for kw in (dict(debug=True), dict(nvtx=True)):
        path = build.build(**kw)
        assert path != ngc.LIB_PATH and os.path.exists(path)
        lib = C.CDLL(path)
        for s in declared_symbols():
            assert hasattr(lib, s), f"{s} missing from {os.path.basename(path)}"
        lib.ngc_version.restype = C.c_int
        assert lib.ngc_version() == ngc.version()
