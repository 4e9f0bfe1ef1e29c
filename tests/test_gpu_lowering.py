"""ekv_lower_sparse_metadata / ekv_reset_tags on the GPU against the lowering oracle: table rows,
lengths, boundaries and flags compared with ==, the tag cross-check on planted disagreements, and
agreement with the tag-scanning ekv_lower_metadata on the state it leaves (Sec. 3.4 / App. B.3)."""
import numpy as np
import pytest
import torch

from oracle import lowering
from gpu_util import require_gpu, dev_i32
from test_oracle_lowering import _random_state

pytestmark = pytest.mark.gpu


def pack_sparse(rows, lens, lists, ranges):
    """The scheduler-side description as ONE int32 host buffer plus the offsets of its parts."""
    blk_start = np.concatenate([[0], np.cumsum([len(x) for x in lists])]).astype(np.int32)
    rng_start = np.concatenate([[0], np.cumsum([len(x) for x in ranges])]).astype(np.int32)
    parts = [np.asarray(rows, np.int32), np.asarray(lens, np.int32), blk_start,
             np.asarray([v for x in lists for v in x], np.int32), rng_start,
             np.asarray([v for x in ranges for ab in x for v in ab], np.int32)]
    offs = np.concatenate([[0], np.cumsum([len(p) for p in parts])])
    return np.concatenate(parts).astype(np.int32), offs


def gpu_lower(b, tags, table, seq_lens, rows, lens, lists, ranges, num_kv_heads=2, head_dim=64):
    nb = len(tags)
    kv = torch.zeros((1, nb, num_kv_heads * 16 * head_dim), dtype=torch.int16, device="cuda")
    pool = b.Pool(kv, kv, torch.from_numpy(tags.copy()).cuda(), num_kv_heads, head_dim)
    d_table, d_sl = torch.from_numpy(table.copy()).cuda(), torch.from_numpy(seq_lens.copy()).cuda()
    batch = b.Batch(d_table, d_sl, True)
    buf, offs = pack_sparse(rows, lens, lists, ranges)
    arena = torch.from_numpy(buf).cuda()                    # one copy for the whole description
    v = [arena[offs[k]:offs[k + 1]] for k in range(6)]
    bounds = torch.full((table.shape[0], 2), 0, dtype=torch.int32, device="cuda")
    flags = torch.full((4,), -1, dtype=torch.int32, device="cuda")
    b.ekv_lower_sparse_metadata(pool, batch, d_sl, v[0], v[1], v[2], v[3], v[4], v[5] if len(v[5]) else None, bounds, flags)
    torch.cuda.synchronize()
    return pool, batch, d_table.cpu().numpy(), d_sl.cpu().numpy(), bounds.cpu().numpy(), flags.cpu().numpy()


@pytest.mark.parametrize("seed", range(8))
def test_lowering_matches_oracle(seed):
    b = require_gpu()
    rs = np.random.default_rng(100 + seed)
    B = int(rs.integers(1, 40))
    tags, lens, lists, modes = _random_state(rs, B=B, max_blocks=70, num_blocks=3000, irregular=seed % 2 == 0)
    ranges = [lowering.ranges_of_modes(m) for m in modes]
    rows = rs.permutation(B + 5)[:B].astype(np.int32)
    table = rs.integers(-5, 0, size=(B + 5, 70)).astype(np.int32)
    sl = np.full(B + 5, -3, np.int32)
    if seed >= 4:                                           # plant disagreements between tags and ranges
        for i in rs.permutation(B)[:3]:
            if len(modes[i]) >= 2:
                tags[lists[i][2 * int(rs.integers(0, len(modes[i]) - 1))]] ^= 1
    o_table, o_sl = table.copy(), sl.copy()
    o_bounds, o_flags = lowering.lower_sparse(o_table, o_sl, tags, rows, lens, lists, ranges)
    pool, batch, g_table, g_sl, g_bounds, g_flags = gpu_lower(b, tags, table, sl, rows, lens, lists, ranges)
    assert np.array_equal(g_table, o_table) and np.array_equal(g_sl, o_sl)
    assert np.array_equal(g_bounds, o_bounds) and np.array_equal(g_flags, o_flags)
    if seed < 4:
        # the tag-scanning lowering must report the same boundaries for the rows in use
        used = torch.from_numpy(np.sort(rows)).cuda().long()
        sub = b.Batch(batch.block_table[used].contiguous(), batch.seq_lens[used].contiguous(), True)
        b2 = torch.zeros((B, 2), dtype=torch.int32, device="cuda")
        f2 = torch.zeros(2, dtype=torch.int32, device="cuda")
        b.ekv_lower_metadata(pool, sub, b2, f2)
        torch.cuda.synchronize()
        assert np.array_equal(b2.cpu().numpy(), g_bounds[np.sort(rows)])
        assert f2.cpu().tolist() == g_flags[:2].tolist()


def test_empty_step_and_no_ranges():
    b = require_gpu()
    tags = np.zeros(64, np.uint8)
    table = np.full((3, 8), -1, np.int32); sl = np.zeros(3, np.int32)
    _, _, g_table, g_sl, g_bounds, g_flags = gpu_lower(b, tags, table, sl, [], [], [], [])
    assert np.array_equal(g_table, table) and g_flags.tolist() == [0, 0, 0, 0]
    _, _, g_table, g_sl, g_bounds, g_flags = gpu_lower(b, tags, table, sl, [2], [40], [[5, 6, 7]], [[]])
    assert g_table[2].tolist() == [5, 6, 7, -1, -1, -1, -1, -1] and g_sl.tolist() == [0, 0, 40]
    assert g_flags.tolist() == [0, 0, 0, 0] and not g_bounds.any()


def test_reset_tags():
    b = require_gpu()
    kv = torch.zeros((1, 50, 2 * 16 * 64), dtype=torch.int16, device="cuda")
    tags = torch.ones(50, dtype=torch.uint8, device="cuda")
    pool = b.Pool(kv, kv, tags, 2, 64)
    ids = np.array([3, 7, 49, 0], np.int32)
    b.ekv_reset_tags(pool, dev_i32(ids))
    torch.cuda.synchronize()
    exp = np.ones(50, np.uint8); exp[ids] = 0
    assert np.array_equal(tags.cpu().numpy(), exp)
