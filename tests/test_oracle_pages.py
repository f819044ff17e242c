"""Pins for the oracle's page bookkeeping (reserve = ADD / growth, release = ABORT / eviction; Sec. 6.1, 6.2):
conservation of pages, stack order, exact counts from the closed form ceil((len+n)/P) - ceil(len/P), and a
brute-force simulation written independently with Python lists."""
import numpy as np
import pytest

import oracle


def simulate(free, P, table, lens, ops):
    """Independent model: python lists, one page at a time."""
    free = list(free)
    table = [list(r) for r in table]
    lens = list(lens)
    for kind, t, n in ops:
        if kind == "reserve":
            have = -(-lens[t] // P)
            want = -(-(lens[t] + n) // P)
            for lp in range(have, want):
                table[t][lp] = free.pop()
        else:
            for lp in range(-(-lens[t] // P)):
                free.append(table[t][lp])
                table[t][lp] = -1
            lens[t] = 0
    return free, table, lens


def test_reserve_and_release_against_list_model():
    rng = np.random.default_rng(1)
    P, T, max_pages, num_pages = 16, 6, 12, 64
    free = rng.permutation(num_pages).astype(np.int32)
    cnt = num_pages
    table = np.full((T, max_pages), -1, np.int32)
    lens = np.zeros(T, np.int32)
    m_free, m_table, m_lens = list(free), table.tolist(), lens.tolist()
    for step in range(30):
        ids = rng.permutation(T)[: rng.integers(1, T + 1)].astype(np.int32)
        if step % 4 == 3:
            cnt = oracle.pages_release(free, cnt, P, table, lens, ids)
            m_free, m_table, m_lens = simulate(m_free, P, m_table, m_lens, [("release", int(t), 0) for t in ids])
        else:
            new = rng.integers(0, 40, size=len(ids)).astype(np.int32)
            new = np.minimum(new, max_pages * P - lens[ids])
            cnt = oracle.pages_reserve(free, cnt, P, table, lens, new, traj_ids=ids)
            m_free, m_table, m_lens = simulate(m_free, P, m_table, m_lens, [("reserve", int(t), int(n)) for t, n in zip(ids, new)])
            lens[ids] += new            # the append that follows a reservation moves the lengths
            for t, n in zip(ids, new):
                m_lens[t] += int(n)
        assert cnt == len(m_free) and list(free[:cnt]) == m_free
        assert table.tolist() == m_table and lens.tolist() == m_lens
        # conservation: every page is either free or owned exactly once
        owned = table[table >= 0]
        assert len(set(owned.tolist()) | set(free[:cnt].tolist())) == num_pages and len(owned) + cnt == num_pages


def test_reserve_counts_follow_the_closed_form_and_take_from_the_top():
    P = 16
    free = np.arange(100, 120, dtype=np.int32)
    table = np.full((3, 8), -1, np.int32)
    table[0, 0] = 7
    lens = np.array([16, 0, 0], np.int32)            # trajectory 0 owns exactly one full page
    cnt = oracle.pages_reserve(free, 20, P, table, lens, np.array([1, 33, 0], np.int32))
    assert cnt == 20 - (1 + 3 + 0)
    assert table[0].tolist()[:3] == [7, 119, -1]     # grows by one page: the top of the stack
    assert table[1].tolist()[:4] == [118, 117, 116, -1]
    assert (table[2] == -1).all()


def test_reserve_refuses_without_side_effects():
    P = 16
    free = np.arange(4, dtype=np.int32)
    table = np.full((2, 3), -1, np.int32)
    lens = np.zeros(2, np.int32)
    t0, f0 = table.copy(), free.copy()
    with pytest.raises(oracle.OracleError):          # needs 5 pages, 4 free
        oracle.pages_reserve(free, 4, P, table, lens, np.array([40, 33], np.int32))
    with pytest.raises(oracle.OracleError):          # 4 pages do not fit a 3-entry row
        oracle.pages_reserve(free, 4, P, table, lens, np.array([49, 0], np.int32))
    assert np.array_equal(table, t0) and np.array_equal(free, f0)


def test_release_then_reserve_reuses_pages_in_stack_order():
    P = 16
    free = np.array([5, 6, 0, 0, 0, 0], np.int32)
    table = np.array([[1, 2, -1], [3, -1, -1]], np.int32)
    lens = np.array([20, 9], np.int32)
    cnt = oracle.pages_release(free, 2, P, table, lens, np.array([1, 0], np.int32))
    assert cnt == 5 and free[:5].tolist() == [5, 6, 3, 1, 2]
    assert (table == -1).all() and lens.tolist() == [0, 0]
    cnt = oracle.pages_reserve(free, cnt, P, table, lens, np.array([17], np.int32), traj_ids=np.array([1], np.int32))
    assert cnt == 3 and table[1].tolist() == [2, 1, -1]


def test_stale_eviction_against_list_model_and_closed_form():
    # Sec. 6.2: with the model at version n, trajectories started before version n - alpha are evicted.  Independent
    # model: python lists and the release model above; closed form: how many go and how many pages come back.
    rng = np.random.default_rng(5)
    P, T, max_pages, num_pages = 16, 40, 6, 300
    for trial in range(20):
        lens = rng.integers(0, max_pages * P + 1, size=T).astype(np.int32)
        lens[rng.integers(0, T, size=6)] = 0                      # empty rows own nothing and are never evicted
        pages = -(-lens // P)
        perm = rng.permutation(num_pages).astype(np.int32)
        table = np.full((T, max_pages), -1, np.int32)
        o = 0
        for t in range(T):
            table[t, :pages[t]] = perm[o:o + pages[t]]
            o += int(pages[t])
        free = np.zeros(num_pages, np.int32)
        cnt = num_pages - o
        free[:cnt] = perm[o:]
        n, alpha = int(rng.integers(3, 9)), int(rng.integers(0, 4))
        sv = rng.integers(0, n + 1, size=T).astype(np.int32)
        sv[rng.integers(0, T, size=5)] = n - alpha                # on the boundary: still inside the window
        stale = [t for t in range(T) if lens[t] > 0 and sv[t] < n - alpha]
        m_free, m_table, m_lens = simulate(free[:cnt], P, table, lens, [("release", t, 0) for t in stale])
        table2, lens2 = table.copy(), lens.copy()
        new_cnt, ids = oracle.pages_evict_stale(free, cnt, P, table2, lens2, sv, n, alpha)
        assert ids.tolist() == stale
        assert new_cnt == cnt + int(pages[stale].sum()) == len(m_free) and free[:new_cnt].tolist() == m_free
        assert table2.tolist() == m_table and lens2.tolist() == m_lens
        assert all(sv[t] >= n - alpha or lens[t] == 0 for t in range(T) if lens2[t] == lens[t])


def test_stale_eviction_boundary_and_all_or_nothing():
    P = 16
    table = np.array([[4, 5, -1], [6, -1, -1], [7, -1, -1], [-1, -1, -1]], np.int32)
    lens = np.array([20, 16, 3, 0], np.int32)
    free = np.array([9, 0, 0, 0, 0, 0], np.int32)
    # version 5, alpha 1: started at 4 stays, started at 3 goes; the empty row (version 0) is not a trajectory
    cnt, ids = oracle.pages_evict_stale(free, 1, P, table, lens, np.array([3, 4, 3, 0], np.int32), 5, 1)
    assert ids.tolist() == [0, 2] and cnt == 4 and free[:4].tolist() == [9, 4, 5, 7]
    assert lens.tolist() == [0, 16, 0, 0] and table.tolist() == [[-1, -1, -1], [6, -1, -1], [-1, -1, -1], [-1, -1, -1]]
    # alpha large enough: nothing goes
    cnt2, ids2 = oracle.pages_evict_stale(free, cnt, P, table, lens, np.array([3, 4, 3, 0], np.int32), 5, 9)
    assert cnt2 == cnt and len(ids2) == 0
    # a stack that cannot take the pages: refused, nothing changes
    small = np.array([1, 0], np.int32)
    t0, l0 = table.copy(), lens.copy()
    with pytest.raises(oracle.OracleError):
        oracle.pages_evict_stale(small, 2, P, table, lens, np.array([0, 0, 0, 0], np.int32), 5, 1)
    assert np.array_equal(table, t0) and np.array_equal(lens, l0) and small.tolist() == [1, 0]
