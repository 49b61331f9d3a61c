"""How the attention kernel divides a launch over its CTAs (host replay; no GPU needed).

Eq. 1 is computed per query tile over key tiles of 128; the kernel lays the key steps of all
query-tile pairs on one line and gives every CTA an equal range of it.  The replay runs the same
code the device roles run to find their segments, so the invariants below are those of a launch.
"""

import ctypes as C

import numpy as np
import pytest


def replay(n_tok, h, h_kv, d, ln, max_ctas):
    from paper_2410_01805_b200 import lib
    n = lib.locret_selftest_attention_split(n_tok, h, h_kv, d, ln, max_ctas, None, 0, None, None)
    assert n >= 0, n
    rows = np.zeros((n, 8), dtype=np.int32)
    u, s = C.c_int32(), C.c_int32()
    assert lib.locret_selftest_attention_split(n_tok, h, h_kv, d, ln, max_ctas, rows.ctypes.data, n,
                                               C.byref(u), C.byref(s)) == n
    return rows, u.value, s.value


def key_tiles(n_tok, h, h_kv, ln):
    """Key tiles per item by the definition: a pair of 128-row query tiles sees the keys up to the last
    row of its lower tile, in tiles of 128, never more than cache + chunk holds."""
    pair = (h // h_kv) % 2 == 0
    n_rb = -(-n_tok // 128)
    out = []
    groups = range(n_rb - 1, -1, -1) if pair else range((n_rb + 1) // 2 - 1, -1, -1)
    for g in groups:
        last_row = g * 128 + 127 if pair else g * 256 + 255
        nk = min((ln + last_row) // 128 + 1, -(-(ln + n_tok) // 128))
        out += [nk] * (h // 2 if pair else h)
    return out


CASES = [
    (3072, 32, 8, 128, 6000, 148),     # the headline launch
    (1024, 32, 32, 96, 16384, 148),    # MHA: row-block pairs, items longer than a CTA's share
    (3072, 32, 8, 128, 0, 148),        # first chunk: only the causal part
    (2048, 32, 8, 128, 6000, 296),
    (200, 4, 2, 64, 300, 7), (129, 3, 3, 96, 1, 5), (64, 8, 1, 128, 0, 148), (512, 8, 2, 64, 1024, 33),
    (10240, 32, 8, 128, 6000, 148),
]


@pytest.mark.parametrize("n_tok,h,h_kv,d,ln,max_ctas", CASES)
def test_every_key_step_is_done_once_and_shares_are_equal(n_tok, h, h_kv, d, ln, max_ctas):
    rows, units, total = replay(n_tok, h, h_kv, d, ln, max_ctas)
    nk = key_tiles(n_tok, h, h_kv, ln)
    assert total == sum(nk) and 1 <= units <= max_ctas
    assert units == max(1, min(max_ctas, total // 4))
    covered = [np.zeros(k, dtype=np.int32) for k in nk]
    per_cta = np.zeros(units, dtype=np.int64)
    for u, item, k0, k1, n, slot, ua, ub in rows:
        assert 0 <= k0 < k1 <= n == nk[item]
        covered[item][k0:k1] += 1
        per_cta[u] += k1 - k0
        assert ua <= u <= ub
        assert (slot == -1) == (k0 == 0 and k1 == n)
        assert (slot == -1) == (ua == ub)
    assert all((c == 1).all() for c in covered)
    assert per_cta.max() - per_cta.min() <= 1 and per_cta.sum() == total
    # CTAs walk the line in order: items ascending, a CTA's segments contiguous
    assert np.all(np.diff(rows[:, 0]) >= 0) and np.all(np.diff(rows[:, 1]) >= 0)


@pytest.mark.parametrize("n_tok,h,h_kv,d,ln,max_ctas", CASES)
def test_pieces_of_an_item_have_distinct_slots_and_the_merge_finds_them(n_tok, h, h_kv, d, ln, max_ctas):
    rows, units, total = replay(n_tok, h, h_kv, d, ln, max_ctas)
    pieces = rows[rows[:, 5] >= 0]
    assert len(set(pieces[:, 5].tolist())) == len(pieces)            # no two pieces share a scratch slot
    assert pieces[:, 5].max(initial=0) < 2 * units
    for item in np.unique(pieces[:, 1]):
        mine = pieces[pieces[:, 1] == item]
        ua, ub = mine[0, 6], mine[0, 7]
        assert list(mine[:, 0]) == list(range(ua, ub + 1))           # one piece per CTA from first to last
        assert mine[0, 2] == 0 and mine[-1, 3] == mine[0, 4]          # together they are the whole item
        assert np.all(mine[1:, 2] == mine[:-1, 3])
    # at most two pieces per CTA: the tail of an item begun earlier and the head of one continued later
    for u in range(units):
        assert np.sum(pieces[:, 0] == u) <= 2


def test_rejects_shapes_the_kernel_does_not_take():
    from paper_2410_01805_b200 import lib
    assert lib.locret_selftest_attention_split(32, 4, 2, 64, 0, 8, None, 0, None, None) == -1      # fewer than 64 tokens
    assert lib.locret_selftest_attention_split(128, 4, 2, 80, 0, 8, None, 0, None, None) == -1     # head_dim
    assert lib.locret_selftest_attention_split(128, 4, 3, 64, 0, 8, None, 0, None, None) == -1
