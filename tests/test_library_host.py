"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares, sizes
buffers consistently and validates arguments before touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2608_30252_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "masw.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b([a-z_][a-z0-9_]*)\s*\(", header)) - {"defined"}
    assert declared == set(binding.EXPORTED_SYMBOLS), declared ^ set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert "sm_100a" in binding.version()


def test_sizes_follow_the_three_region_layout(lib):
    cfg = binding.MaswConfig(16, 1, 32, 8, 64, 2048, 128, 128, 4, rollback=16, max_slots=8200, gamma_max=8)
    arena, ws = binding.masw_sizes(cfg)
    ring = (128 + 16 + 8 + 63) // 64 * 64
    assert arena == 16 * 2 * 1 * 8 * (128 + 8200 + ring) * 64 * 2
    assert ws > 0 and ws % 256 == 0
    # batch scales the arena linearly
    cfg4 = binding.MaswConfig(16, 4, 32, 8, 64, 2048, 128, 128, 4, rollback=16, max_slots=8200, gamma_max=8)
    assert binding.masw_sizes(cfg4)[0] == 4 * arena


def test_prefill_slot_count_is_the_paper_s_boundary_rule(lib, golden_dir):
    """draft_prefill_slots (host only): floor((P - S) / r) slots inside a prefix of P tokens (Section 4.2), checked
    on the paper's constants and against the oracle's count."""
    from oracle import prefill as opf
    rows = [l.split() for l in open(os.path.join(golden_dir, "memory_sizes.txt")) if l[0] != "#" and l.strip()]
    for P, S, W, r, slots, _ in (map(int, x) for x in rows):
        c = binding.MaswConfig(1, 1, 8, 2, 64, 512, S, W, r, rollback=16, max_slots=slots, gamma_max=4).to_c()
        assert lib.draft_prefill_slots(C.byref(c), P) == slots == opf.n_prefill_slots(P, S, r)
    c = binding.MaswConfig(1, 1, 8, 2, 64, 512, 8, 16, 4, max_slots=4).to_c()
    assert [lib.draft_prefill_slots(C.byref(c), P) for P in (0, 7, 8, 11, 12, 13, 16)] == [0, 0, 0, 0, 1, 1, 2]
    assert lib.draft_prefill_slots(None, 5) == -1 and lib.draft_prefill_slots(C.byref(c), -1) == -1


@pytest.mark.parametrize("field,value", [("head_dim", 96), ("n_kv_heads", 3), ("window", 0), ("d_model", 12),
                                         ("gamma_max", 0), ("batch", 0), ("softmax_scale", -1.0)])
def test_bad_configs_are_rejected_with_einval(lib, field, value):
    cfg = binding.MaswConfig(2, 1, 8, 2, 64, 512, 0, 64, 16, max_slots=64, gamma_max=4)
    setattr(cfg, field, value)
    with pytest.raises(binding.MaswError) as ei:
        binding.masw_sizes(cfg)
    assert ei.value.code == binding.MASW_EINVAL
    assert binding.load().masw_last_error()


def test_group_times_rows_limit(lib):
    cfg = binding.MaswConfig(1, 1, 32, 2, 64, 2048, 0, 64, 16, max_slots=64, gamma_max=4)   # G = 16, 5 rows -> 80
    with pytest.raises(binding.MaswError):
        binding.masw_sizes(cfg)


def test_verify_and_accept_validate_before_launch(lib):
    desc = binding.masw_kv_desc(0x1000, 0x2000, 2 * 128 * 64, 128 * 64, 128, 1, 8, 2, 96, 64, 0x3000, 0.0)
    rc = lib.verify_attend(C.byref(desc), C.c_void_p(0x4000), 4, C.c_void_p(0x5000), None, None, C.c_void_p(0x6000), 1 << 20, None)
    assert rc == binding.MASW_EINVAL
    desc.head_dim = 128
    rc = lib.verify_attend(C.byref(desc), C.c_void_p(0x4001), 4, C.c_void_p(0x5000), None, None, C.c_void_p(0x6000), 1 << 20, None)
    assert rc == binding.MASW_EALIGN
    rc = lib.verify_attend(C.byref(desc), C.c_void_p(0x4000), 40, C.c_void_p(0x5000), None, None, C.c_void_p(0x6000), 1 << 20, None)
    assert rc == binding.MASW_EINVAL            # 40 rows x group 4 > 64
    rc = lib.verify_attend(C.byref(desc), C.c_void_p(0x4000), 4, C.c_void_p(0x5000), None, None, C.c_void_p(0x6000), 16, None)
    assert rc == binding.MASW_ECAPACITY
    assert lib.verify_workspace_bytes(C.byref(desc), 4) > 0
    assert lib.accept_workspace_bytes(2, 5, 32000) > 0
    rc = lib.accept_reject(C.c_void_p(0x1000), None, C.c_void_p(0x2000), None, 1, 4, 100, 1.0, C.c_void_p(0x3000),
                           C.c_void_p(0x4000), None, C.c_void_p(0x5000), 1 << 16, None)
    assert rc == binding.MASW_EINVAL            # sampling without draft logits / uniforms


def test_sampling_vocab_bound_and_no_developer_hooks_in_the_product_library(lib):
    """temperature > 0 keeps 64-bit weight sums: a vocabulary of 2^17 or more is refused before any launch (greedy
    has no such bound).  The product library exports none of the developer build's hooks."""
    args = lambda V, temp: (C.c_void_p(0x1000), C.c_void_p(0x1100), C.c_void_p(0x2000), C.c_void_p(0x2100), 1, 4, V, temp,
                            C.c_void_p(0x3000), C.c_void_p(0x4000), None)
    assert lib.accept_reject(*args(131072, 1.0), C.c_void_p(0x5000), 16, None) == binding.MASW_EINVAL
    assert "vocab" in lib.masw_last_error().decode()
    assert lib.accept_reject(*args(131071, 1.0), C.c_void_p(0x5000), 16, None) == binding.MASW_ECAPACITY   # passes the bound, fails on the tiny workspace
    assert lib.accept_reject(*args(200000, 0.0), C.c_void_p(0x5000), 16, None) == binding.MASW_ECAPACITY
    assert lib.accept_reject_static(*args(131072, 1.0), None) == binding.MASW_EINVAL
    for name in ("masw_debug_set_trace", "masw_debug_set_wait", "masw_debug_set_flags", "masw_debug_set_verify_legacy"):
        assert not hasattr(lib, name), name


def test_paged_verify_and_prefill_validate_before_launch(lib):
    """Bad arguments of the two newer entry points are refused on the host (fake pointers are never touched)."""
    vp, i32, sz = C.c_void_p, C.c_int, C.c_size_t
    lib.verify_attend_paged.argtypes = [C.POINTER(binding.masw_paged_kv_desc), vp, i32, vp, vp, vp, vp, sz, vp]
    lib.verify_paged_workspace_bytes.argtypes = [C.POINTER(binding.masw_paged_kv_desc), i32]
    lib.verify_paged_workspace_bytes.restype = sz
    d = binding.masw_paged_kv_desc(0x1000, 0x2000, 0x3000, 64, 16, 1, 8, 2, 64, 0x4000, 0.0)
    call = lambda q=0x5000, T=4, ws=1 << 24: lib.verify_attend_paged(C.byref(d), vp(q), T, vp(0x6000), None, None, vp(0x7000), ws, None)
    assert call() == binding.MASW_EINVAL                      # head_dim 64: the paged path is the head_dim-128 kernel
    d.head_dim = 128
    assert call(q=0x5008) == binding.MASW_EALIGN
    assert call(T=20) == binding.MASW_EINVAL                  # 20 rows x group 4 > 64
    assert call(ws=64) == binding.MASW_ECAPACITY
    assert lib.verify_paged_workspace_bytes(C.byref(d), 4) > 0
    d.page_table = None
    assert call() == binding.MASW_EINVAL
    lib.draft_prefill_attend.argtypes = [vp, i32, C.POINTER(binding.masw_kv_desc), vp, i32, vp, vp, vp, i32, vp]
    kv = binding.masw_kv_desc(0x1000, 0x2000, 2 * 128 * 64, 128 * 64, 64, 1, 8, 2, 64, 128, None, 0.0)
    assert lib.draft_prefill_attend(None, 0, C.byref(kv), vp(0x5000), 16, vp(0x6000), None, None, 0, None) == binding.MASW_EINVAL


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "libmasw.so"))
    with pytest.raises(FileNotFoundError):
        binding.load()
