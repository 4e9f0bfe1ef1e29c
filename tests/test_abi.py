"""The C-ABI library loads without a GPU and exports every entry point include/ekv.h declares;
host-side argument checks return error codes before anything is launched."""
import ctypes as C
import os
import re

import pytest

from paper_2609_33536_b200 import binding, build as ekv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    ekv_build.build()
    return binding.load()


def _declared():
    names = set()
    for header in ("ekv.h", "ekv_controller.h"):
        text = open(os.path.join(ROOT, "include", header)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(ekv_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    from paper_2609_33536_b200 import controller
    assert set(binding.EXPORTS) | set(controller.EXPORTS) == set(names)
    assert len(names) >= 30
    for n in names:
        assert hasattr(lib, n), n


def test_struct_sizes_match_header():
    assert C.sizeof(binding.ekv_pool) == 56
    assert C.sizeof(binding.ekv_batch) == 32


def test_status_strings(lib):
    assert lib.ekv_status_string(0) == b"ok"
    assert b"workspace" in lib.ekv_status_string(-3)
    assert lib.ekv_version() >= 100


def test_host_side_argument_checks(lib):
    """No GPU: all of these must be rejected on the host before any launch."""
    pool = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 2, 64, 16, 1, 0, 8 * 2 * 16 * 64 * 2)
    batch = binding.ekv_batch(0x4000, 0x5000, 2, 4, 0, 0)
    dec = lambda p, b, q=0x6000, o=0x7000, hq=8, ms=64: lib.ekv_attn_decode(
        C.byref(p), 0, C.byref(b), q, o, hq, 0.125, ms, None, 0, None)
    assert dec(pool, batch, q=None) == -1                        # null q
    assert dec(pool, batch, hq=7) == -1                          # heads not a multiple of kv heads
    assert dec(pool, batch, hq=32) == -2                         # 16 query heads per kv head
    assert dec(pool, batch, ms=65) == -1                         # max_seq_len beyond the table
    bad = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 2, 96, 16, 1, 0, 1 << 20)
    assert dec(bad, batch) == -2                                 # head_dim 96
    bad = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 2, 64, 32, 1, 0, 1 << 20)
    assert dec(bad, batch) == -2                                 # page size 32
    bad = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 2, 64, 16, 1, 0, 100)
    assert dec(bad, batch) == -1                                 # layer stride too small
    assert lib.ekv_attn_decode(C.byref(pool), 3, C.byref(batch), 0x6000, 0x7000, 8, 0.125, 64, None, 0, None) == -1
    assert lib.ekv_downgrade(C.byref(pool), C.byref(batch), -1, None, None, None, None, None, None, None) == -1
    assert lib.ekv_downgrade(C.byref(pool), C.byref(batch), 0, None, None, None, None, None, None, None) == 0
    assert lib.ekv_downgrade(C.byref(pool), C.byref(batch), 1, 0x10, 0x20, 0x100, None, None, 0x30, None) == -1
    assert lib.ekv_refine(C.byref(pool), C.byref(batch), 1, 0x10, 0x20, None, 0x100, 0x200, 0x30, None) == -1
    assert lib.ekv_set_option(b"no_such_option", 1) == -1
    assert lib.ekv_set_option(b"decode_chunk_tokens", 0) == 0


def test_workspace_sizing(lib):
    pool = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 8, 128, 16, 1, 0, 1 << 30)
    assert lib.ekv_attn_workspace_bytes(C.byref(pool), 2, 32, 200, 0) == 0          # single split
    lib.ekv_set_option(b"decode_chunk_tokens", 1024)
    n = lib.ekv_attn_workspace_bytes(C.byref(pool), 64, 32, 8192, 0)
    rows = 64 * 32 * 8
    assert n >= rows * 128 * 4 + rows * 4
    # a too-small workspace is refused on the host
    batch = binding.ekv_batch(0x4000, 0x5000, 64, 512, 1, 0)
    assert lib.ekv_attn_decode(C.byref(pool), 0, C.byref(batch), 0x6000, 0x7000, 32, 0.1, 8192, 0x100, n - 1, None) == -3
    lib.ekv_set_option(b"decode_chunk_tokens", 0)


def test_argument_checks_of_the_later_entry_points(lib):
    """Lowering, tag reset, the no-workspace decode and the options: refused on the host, no launch."""
    pool = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 2, 64, 16, 1, 0, 8 * 2 * 16 * 64 * 2)
    batch = binding.ekv_batch(0x4000, 0x5000, 2, 4, 1, 0)
    low = lambda n=1, sl=0x10, lens=0x20, bs=0x30, ids=0x40, rs=0x50, bounds=0x60, flags=0x70, row_of=None: \
        lib.ekv_lower_sparse_metadata(C.byref(pool), C.byref(batch), sl, n, row_of, lens, bs, ids, rs, None, bounds, flags, None)
    assert low(n=-1) == -1
    assert low(sl=None) == -1 and low(bounds=None) == -1 and low(flags=None) == -1
    assert low(lens=None) == -1 and low(bs=None) == -1 and low(ids=None) == -1 and low(rs=None) == -1
    assert low(n=3) == -1                                        # more requests than table rows, no row_of
    no_tags = binding.ekv_pool(0x1000, 0x2000, None, 8, 2, 64, 16, 1, 0, 8 * 2 * 16 * 64 * 2)
    assert lib.ekv_lower_sparse_metadata(C.byref(no_tags), C.byref(batch), 0x10, 1, None, 0x20, 0x30, 0x40, 0x50, None,
                                         0x60, 0x70, None) == -1
    assert lib.ekv_reset_tags(C.byref(pool), None, 3, None) == -1
    assert lib.ekv_reset_tags(C.byref(pool), None, 0, None) == 0
    assert lib.ekv_reset_tags(C.byref(no_tags), 0x10, 1, None) == -1
    # the no-workspace decode: argument errors first, then the size of its fixed array
    assert lib.ekv_attn_decode_noalloc(None, 0, C.byref(batch), 0x6000, 0x7000, 8, 0.125, 64, None) == -1
    assert lib.ekv_attn_decode_noalloc(C.byref(pool), 0, C.byref(batch), 0x6000, 0x7000, 0, 0.125, 64, None) == -1
    big = binding.ekv_pool(0x1000, 0x2000, 0x3000, 1 << 20, 8, 128, 16, 1, 0, (1 << 20) * 8 * 16 * 128 * 2)
    bb = binding.ekv_batch(0x4000, 0x5000, 256, 1 << 14, 1, 0)
    lib.ekv_set_option(b"decode_chunk_tokens", 64)
    assert lib.ekv_attn_workspace_bytes(C.byref(big), 256, 64, 1 << 18, 0) > lib.ekv_attn_decode_noalloc_max_bytes()
    assert lib.ekv_attn_decode_noalloc(C.byref(big), 0, C.byref(bb), 0x6000, 0x7000, 64, 0.1, 1 << 18, None) == -3
    lib.ekv_set_option(b"decode_chunk_tokens", 0)
    for name, bad in ((b"decode_two_term", 3), (b"prefill_p_terms", 3), (b"decode_staging", 3), (b"attn_out_f32", 2),
                      (b"decode_merge_slices", 3), (b"decode_variant", 2), (b"prefill_variant", 2)):
        assert lib.ekv_set_option(name, bad) == -1, name
        assert lib.ekv_set_option(name, 0) == 0, name


def test_split_size_rule(lib):
    """The automatic split size, read back through the workspace size (partials = rows x splits x (D + 1) floats):
    small launches get one balanced wave of at most two CTAs per SM, large ones splits of at most 3200 tokens."""
    pool = binding.ekv_pool(0x1000, 0x2000, 0x3000, 8, 8, 128, 16, 1, 0, 1 << 30)

    def splits(batch, max_len, hq=32):
        n = lib.ekv_attn_workspace_bytes(C.byref(pool), batch, hq, max_len, 0)
        rows = batch * hq
        return 1 if n == 0 else round(n / (rows * 129 * 4))
    # without a GPU the SM count falls back to 148
    assert splits(64, 8192) == 3                                 # 3200-token splits
    assert splits(8, 8192) == 4                                  # 64 units x 4 = 256 CTAs <= 296
    assert splits(4, 32768) == 9                                 # 32 units x 9 = 288 CTAs
    assert splits(1, 8192) == 32                                 # floor of 256 tokens
    assert splits(256, 16384) == 6                               # capped at 3200 tokens: ceil(16384 / 3200)
