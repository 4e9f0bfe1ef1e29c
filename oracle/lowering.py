"""TEST INFRASTRUCTURE. Plain restatement of the worker-side metadata lowering (Sec. 3.4; App. B.3):
the scheduler describes a scheduled request by its length, its logical -> physical block list and
a sparse, sorted list of BASE pair ranges; the worker needs dense table rows, lengths, the two
mode boundaries of the structured path (Sec. 3.2), the batch flags, and a check of the ranges
against the per-block tags. Pure-Python loops, one request and one pair at a time."""
import numpy as np

TARGET, BASE = 0, 1


def lower_sparse(block_table, seq_lens, tags, rows, lens, block_lists, range_lists):
    """block_table [B][max_blocks] and seq_lens [B] are updated in place (rows named in `rows`).
    Returns (boundaries [B][2] with untouched rows zero, flags [4])."""
    B = block_table.shape[0]
    boundaries = np.zeros((B, 2), dtype=np.int32)
    any_base = any_irregular = 0
    n_bad = 0
    first_bad = None
    n_req = len(rows)
    for i in range(n_req):
        row, ids, ranges = int(rows[i]), list(block_lists[i]), [tuple(r) for r in range_lists[i]]
        for lb, phys in enumerate(ids):
            block_table[row, lb] = phys
        seq_lens[row] = lens[i]
        if ranges:
            any_base = 1
            boundaries[row] = (ranges[0][0], ranges[-1][1])
            for (a0, a1), (b0, b1) in zip(ranges[:-1], ranges[1:]):
                if b0 > a1:                     # a TARGET pair between two BASE runs
                    any_irregular = 1
        bad_here = 0
        for p in range((len(ids) + 1) // 2):
            in_range = any(a <= p < b for a, b in ranges)
            id0 = ids[2 * p]
            id1 = ids[2 * p + 1] if 2 * p + 1 < len(ids) else None
            ok = 0 <= id0 < len(tags) and (id1 is None or id1 < len(tags))
            if ok:
                tag_base = tags[id0] == BASE
                ok = (tag_base == in_range) and ((id1 == id0) if in_range else (id1 != id0))
            if not ok:
                bad_here += 1
        if bad_here:
            n_bad += bad_here
            if first_bad is None:
                first_bad = i
    flags = np.array([any_base, any_irregular, n_bad, 0 if first_bad is None else n_req - first_bad], dtype=np.int32)
    return boundaries, flags


def ranges_of_modes(pair_is_base):
    """Dense per-pair booleans -> the sorted list of maximal [first, one past last) BASE runs."""
    out, start = [], None
    for p, b in enumerate(list(pair_is_base) + [False]):
        if b and start is None:
            start = p
        if not b and start is not None:
            out.append((start, p))
            start = None
    return out
