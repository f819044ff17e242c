"""Pins for the CPU oracle: closed forms, invariants, an independent dense routine, brute force.

The paper gives no worked numeric example of the engine step (Sec. 6.1 treats it as a black
box), so the oracle is pinned to what mathematics fixes.  Each test is chosen so that a plausible
slip in the oracle (dropped scale, wrong sign, pos/P vs pos%P swapped, wrong head mapping,
off-by-one in the causal count, missing max subtraction, stale-slot reads) fails at least one.
"""
import math
import os

import numpy as np
import pytest

import oracle
from paging import bits_to_f64, pack_pages, to_bf16_bits

D = 128
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_bits(rng, *shape, scale=1.0):
    return to_bf16_bits(rng.standard_normal(shape) * scale)


def dense_attention(q_bits, K_bits, V_bits, scale, g):
    """Independent routine: unpaged numpy float64 softmax(q K^T) V for one trajectory.
    q [Hq][D], K/V [L][Hkv][D]  ->  out [Hq][D], lse [Hq]."""
    q = bits_to_f64(q_bits)
    K = bits_to_f64(K_bits)
    V = bits_to_f64(V_bits)
    Hq = q.shape[0]
    out = np.zeros((Hq, q.shape[1]))
    lse = np.zeros(Hq)
    for hq in range(Hq):
        h = hq // g
        s = np.float64(np.float32(scale)) * (K[:, h, :] @ q[hq])
        p = np.exp(s - s.max())
        out[hq] = (p[:, None] * V[:, h, :]).sum(0) / p.sum()
        lse[hq] = s.max() + math.log(p.sum())
    return out, lse


def run_decode(K_list, V_list, q_bits, scale, P, rng=None, **pack_kw):
    Hkv = K_list[0].shape[1]
    kp, vp, table, lens = pack_pages(K_list, V_list, P, Hkv, K_list[0].shape[2], rng=rng, **pack_kw)
    return oracle.decode_attn(kp, vp, table, lens, q_bits, scale)


# ---- P1: single key ---------------------------------------------------------------------------
def test_single_key_returns_v_exactly():
    rng = np.random.default_rng(1)
    K = [rand_bits(rng, 1, 2, D)]
    V = [rand_bits(rng, 1, 2, D)]
    q = rand_bits(rng, 1, 8, D)
    out, lse = run_decode(K, V, q, 0.25, 16)
    for hq in range(8):
        h = hq // 4
        assert np.array_equal(out[0, hq], bits_to_f64(V[0][0, h]))
        s0 = 0.25 * float(bits_to_f64(q[0, hq]) @ bits_to_f64(K[0][0, h]))
        assert lse[0, hq] == pytest.approx(s0, rel=1e-14, abs=1e-14)


# ---- P2: uniform keys -> mean of v --------------------------------------------------------------
@pytest.mark.parametrize("L", [2, 16, 17, 100])
def test_uniform_keys_give_mean_of_v(L):
    rng = np.random.default_rng(2)
    k1 = rand_bits(rng, 1, 2, D)
    K = [np.repeat(k1, L, axis=0)]
    V = [rand_bits(rng, L, 2, D)]
    q = rand_bits(rng, 1, 4, D)
    out, lse = run_decode(K, V, q, 0.1, 16, rng=rng)
    for hq in range(4):
        h = hq // 2
        np.testing.assert_allclose(out[0, hq], bits_to_f64(V[0][:, h]).mean(0), rtol=1e-13, atol=1e-14)
        s = np.float64(np.float32(0.1)) * float(bits_to_f64(q[0, hq]) @ bits_to_f64(k1[0, h]))
        assert lse[0, hq] == pytest.approx(s + math.log(L), rel=1e-13)


# ---- P3: two-key closed form (golden constants) -------------------------------------------------
def test_two_key_closed_form_matches_golden():
    gold = {}
    with open(os.path.join(GOLDEN, "two_key_closed_form.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                gold[k] = float(v)
    rng = np.random.default_rng(3)
    e0 = np.zeros(D, dtype=np.float32)
    e0[0] = 1.0
    K = [to_bf16_bits(np.stack([np.zeros(D, np.float32), e0])[:, None, :])]
    V = [rand_bits(rng, 2, 1, D)]
    q = to_bf16_bits(e0[None, None, :])
    out, lse = run_decode(K, V, q, 1.0, 16)
    v = bits_to_f64(V[0][:, 0])
    np.testing.assert_allclose(out[0, 0], gold["w0"] * v[0] + gold["w1"] * v[1], rtol=1e-14, atol=1e-15)
    assert lse[0, 0] == pytest.approx(gold["lse"], rel=1e-15)
    # the scale multiplies the score: scale 2 -> scores {0, 2}
    out2, lse2 = run_decode(K, V, q, 2.0, 16)
    assert lse2[0, 0] == pytest.approx(math.log(1 + math.exp(2.0)), rel=1e-15)


# ---- P4: constant V ---------------------------------------------------------------------------
def test_constant_v_is_returned_for_any_keys():
    rng = np.random.default_rng(4)
    L = 75
    c = rand_bits(rng, 1, 2, D)
    K = [rand_bits(rng, L, 2, D, scale=3.0)]
    V = [np.repeat(c, L, axis=0)]
    q = rand_bits(rng, 1, 6, D)
    out, _ = run_decode(K, V, q, 0.3, 16, rng=rng)
    for hq in range(6):
        np.testing.assert_allclose(out[0, hq], bits_to_f64(c[0, hq // 3]), rtol=1e-13)


# ---- P5: needle -------------------------------------------------------------------------------
@pytest.mark.parametrize("needle", [0, 15, 16, 47, 48, 63])
def test_needle_dominates(needle):
    rng = np.random.default_rng(5)
    L = 64
    Kf = rng.standard_normal((L, 1, D)).astype(np.float32) * 0.05
    qf = np.zeros((1, 1, D), np.float32)
    qf[0, 0, 3] = 8.0
    Kf[:, 0, 3] = 0.0
    Kf[needle, 0, 3] = 8.0                      # score 64 * 0.5 = 32 above the rest
    K = [to_bf16_bits(Kf)]
    V = [rand_bits(rng, L, 1, D)]
    out, _ = run_decode(K, V, to_bf16_bits(qf), 0.5, 16, rng=rng)
    np.testing.assert_allclose(out[0, 0], bits_to_f64(V[0][needle, 0]), atol=L * math.exp(-32.0) * 8)


# ---- P6: shift invariance -----------------------------------------------------------------------
def test_score_shift_changes_only_lse():
    rng = np.random.default_rng(6)
    L = 40
    Kf = np.round(rng.standard_normal((L, 2, D)) * 4) / 8          # multiples of 1/8: exact in bf16
    qf = np.round(rng.standard_normal((1, 4, D)) * 4) / 8
    qf[0, :, 0] = 2.0
    K0 = to_bf16_bits(Kf)
    Kf2 = Kf.copy()
    Kf2[:, :, 0] += 4.0                                             # still exact
    K1 = to_bf16_bits(Kf2)
    assert np.array_equal(bits_to_f64(K1), Kf2)
    V = [rand_bits(rng, L, 2, D)]
    q = to_bf16_bits(qf)
    o0, l0 = run_decode([K0], V, q, 0.125, 16)
    o1, l1 = run_decode([K1], V, q, 0.125, 16)
    np.testing.assert_allclose(o1, o0, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(l1 - l0, 0.125 * 2.0 * 4.0, rtol=1e-13)


def test_large_scores_do_not_overflow():
    # scores near 3e4: without the max subtraction exp overflows to inf and out becomes NaN
    L = 8
    Kf = np.zeros((L, 1, D), np.float32)
    Kf[:, 0, 0] = 128.0 + np.arange(L)
    qf = np.zeros((1, 1, D), np.float32)
    qf[0, 0, 0] = 256.0
    rng = np.random.default_rng(60)
    V = [rand_bits(rng, L, 1, D)]
    out, lse = run_decode([to_bf16_bits(Kf)], V, to_bf16_bits(qf), 1.0, 16)
    assert np.all(np.isfinite(out)) and np.all(np.isfinite(lse))
    w = np.exp(256.0 * (np.arange(L) - (L - 1.0)))
    np.testing.assert_allclose(out[0, 0], (w[:, None] * bits_to_f64(V[0][:, 0])).sum(0) / w.sum(), rtol=1e-13)


# ---- P7 / P8 / P9: paging invariances and agreement with unpaged dense ---------------------------
def make_case(rng, lens, Hq, Hkv):
    K = [rand_bits(rng, L, Hkv, D) for L in lens]
    V = [rand_bits(rng, L, Hkv, D) for L in lens]
    q = rand_bits(rng, len(lens), Hq, D)
    return K, V, q


def test_page_permutation_is_bit_invariant():
    rng = np.random.default_rng(7)
    K, V, q = make_case(rng, [1, 16, 33, 100, 64], 8, 2)
    ref = run_decode(K, V, q, 0.09, 16)
    for s in range(3):
        got = run_decode(K, V, q, 0.09, 16, rng=np.random.default_rng(100 + s), spare=7)
        assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


@pytest.mark.parametrize("P", [1, 16, 32, 64, 128])
def test_page_size_is_bit_invariant(P):
    rng = np.random.default_rng(8)
    K, V, q = make_case(rng, [5, 64, 65, 127, 128], 4, 4)
    ref = run_decode(K, V, q, 0.2, 128)          # every trajectory in a single page
    got = run_decode(K, V, q, 0.2, P, rng=rng)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])


@pytest.mark.parametrize("Hq,Hkv", [(8, 2), (28, 4), (16, 1), (4, 4)])
def test_equals_unpaged_dense(Hq, Hkv):
    rng = np.random.default_rng(9)
    lens = [1, 2, 15, 16, 17, 31, 32, 33, 200]
    K, V, q = make_case(rng, lens, Hq, Hkv)
    scale = 1.0 / math.sqrt(D)
    out, lse = run_decode(K, V, q, scale, 16, rng=rng)
    for t in range(len(lens)):
        o, l = dense_attention(q[t], K[t], V[t], scale, Hq // Hkv)
        np.testing.assert_allclose(out[t], o, rtol=1e-12, atol=1e-13)
        np.testing.assert_allclose(lse[t], l, rtol=1e-12, atol=1e-12)


# ---- P10: split consistency (the combine formula) ------------------------------------------------
@pytest.mark.parametrize("cuts", [[0, 50, 131], [0, 1, 2, 131], [0, 16, 32, 48, 64, 131], [0, 130, 131], [0, 0, 131]])
def test_parts_combine_to_whole(cuts):
    rng = np.random.default_rng(10)
    L = 131
    K, V, q = make_case(rng, [L], 8, 2)
    kp, vp, table, lens = pack_pages(K, V, 16, 2, D, rng=rng)
    whole_o, whole_l = oracle.decode_attn(kp, vp, table, lens, q, 0.11)
    po, pl = [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, l = oracle.attend_rows(kp, vp, table, [0], [b], q, 0.11, row_begin=[a])
        po.append(o[0])
        pl.append(l[0])
    co, cl = oracle.lse_combine(np.stack(po), np.stack(pl))
    np.testing.assert_allclose(co, whole_o[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(cl, whole_l[0], rtol=1e-13)


def test_combine_two_part_closed_form():
    # parts with lse {0, ln 3} and outs {a, b} -> (a + 3 b) / 4, lse = ln 4
    a = np.arange(8, dtype=np.float64)
    b = -np.ones(8)
    o, l = oracle.lse_combine(np.stack([a, b])[:, None, :], np.array([[0.0], [math.log(3.0)]]))
    np.testing.assert_allclose(o[0], (a + 3 * b) / 4, rtol=1e-15)
    assert l[0] == pytest.approx(math.log(4.0), rel=1e-15)
    # an empty part (lse = -inf) is ignored
    o2, l2 = oracle.lse_combine(np.stack([a, b, 7 * a])[:, None, :], np.array([[0.0], [math.log(3.0)], [-np.inf]]))
    np.testing.assert_allclose(o2[0], o[0], rtol=1e-15)
    assert l2[0] == l[0]


def test_empty_range_gives_zero_and_minus_inf():
    rng = np.random.default_rng(11)
    K, V, q = make_case(rng, [20], 2, 1)
    kp, vp, table, lens = pack_pages(K, V, 16, 1, D)
    o, l = oracle.attend_rows(kp, vp, table, [0], [0], q, 1.0)
    assert np.all(o == 0) and np.all(np.isneginf(l))


# ---- P11: chunk == sequential (append 1, decode) ---------------------------------------------------
def test_chunk_equals_sequential_decode():
    rng = np.random.default_rng(12)
    P, Hq, Hkv = 16, 4, 2
    prior = [30, 0, 16]
    n_new = [21, 5, 1]
    K, V, _ = make_case(rng, [a + b for a, b in zip(prior, n_new)], Hq, Hkv)
    # pools holding only the prior context, table sized for prior + chunk
    mp = max((a + b + P - 1) // P for a, b in zip(prior, n_new))
    Kp = [K[t][:prior[t]] for t in range(3)]
    Vp = [V[t][:prior[t]] for t in range(3)]
    kp, vp, table, lens = pack_pages(Kp, Vp, P, Hkv, D, rng=None, spare=12, max_pages=mp)
    # give every trajectory the pages it will grow into (take them from the spare ones)
    nxt = int(table.max()) + 1
    for t in range(3):
        for lp in range((prior[t] + P - 1) // P, (prior[t] + n_new[t] + P - 1) // P):
            table[t, lp] = nxt
            nxt += 1
    indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    k_new = np.concatenate([K[t][prior[t]:] for t in range(3)])
    v_new = np.concatenate([V[t][prior[t]:] for t in range(3)])
    q = rand_bits(rng, int(indptr[-1]), Hq, D)
    # (a) one chunk call
    kc, vc = kp.copy(), vp.copy()
    after = oracle.kv_append(kc, vc, table, lens, indptr, k_new, v_new)
    assert list(after) == [a + b for a, b in zip(prior, n_new)]
    oc, lc = oracle.obs_chunk_attn(kc, vc, table, after, indptr, q, 0.13)
    # (b) token by token
    ks, vs = kp.copy(), vp.copy()
    cur = lens.copy()
    for t in range(3):
        for j in range(n_new[t]):
            r = indptr[t] + j
            cur = oracle.kv_append(ks, vs, table, cur, np.array([0, 1], np.int32), k_new[r:r + 1], v_new[r:r + 1],
                                   traj_ids=np.array([t], np.int32))
            o1, l1 = oracle.decode_attn(ks, vs, table, cur, q[r:r + 1], 0.13, traj_ids=np.array([t], np.int32))
            assert np.array_equal(o1[0], oc[r]) and np.array_equal(l1[0], lc[r])
    assert np.array_equal(ks, kc) and np.array_equal(vs, vc)
    # (c) and against the independent dense routine with an explicit causal count
    for t in range(3):
        for j in range(n_new[t]):
            c = prior[t] + j + 1
            o, l = dense_attention(q[indptr[t] + j], K[t][:c], V[t][:c], 0.13, Hq // Hkv)
            np.testing.assert_allclose(oc[indptr[t] + j], o, rtol=1e-12, atol=1e-13)


def test_chunk_first_row_of_fresh_trajectory_sees_only_itself():
    rng = np.random.default_rng(13)
    K, V, _ = make_case(rng, [9], 2, 1)
    kp, vp, table, lens = pack_pages(K, V, 16, 1, D)
    q = rand_bits(rng, 9, 2, D)
    o, _ = oracle.obs_chunk_attn(kp, vp, table, lens, np.array([0, 9], np.int32), q, 1.0)
    assert np.array_equal(o[0, 0], bits_to_f64(V[0][0, 0]))
    # subset evaluation agrees with full evaluation
    o_sub, _ = oracle.obs_chunk_attn(kp, vp, table, lens, np.array([0, 9], np.int32), q, 1.0, rows=[8, 3])
    assert np.array_equal(o_sub[0], o[8]) and np.array_equal(o_sub[1], o[3])


# ---- P12: GQA head mapping ---------------------------------------------------------------------
def test_gqa_group_mapping():
    rng = np.random.default_rng(14)
    L, Hq, Hkv = 50, 6, 2
    K, V, q = make_case(rng, [L], Hq, Hkv)
    q[0, 1] = q[0, 0]          # same group (heads 0..2 -> kv head 0)
    q[0, 3] = q[0, 0]          # other group
    out, _ = run_decode(K, V, q, 0.1, 16)
    assert np.array_equal(out[0, 0], out[0, 1])
    assert not np.allclose(out[0, 0], out[0, 3])
    # poisoning kv head 1 must leave heads 0..2 untouched and break heads 3..5
    K2 = [K[0].copy()]
    K2[0][:, 1, :] = 0x7FC0
    out2, _ = run_decode(K2, V, q, 0.1, 16)
    assert np.array_equal(out2[0, :3], out[0, :3])
    assert np.all(np.isnan(out2[0, 3:]))


# ---- P13: duplication --------------------------------------------------------------------------
def test_duplicated_context():
    rng = np.random.default_rng(15)
    K, V, q = make_case(rng, [37], 4, 2)
    o1, l1 = run_decode(K, V, q, 0.2, 16)
    K2 = [np.concatenate([K[0], K[0]])]
    V2 = [np.concatenate([V[0], V[0]])]
    o2, l2 = run_decode(K2, V2, q, 0.2, 16)
    np.testing.assert_allclose(o2, o1, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(l2, l1 + math.log(2.0), rtol=1e-13)


# ---- P14: append round trip ----------------------------------------------------------------------
@pytest.mark.parametrize("P", [16, 64])
def test_append_round_trip_touches_nothing_else(P):
    rng = np.random.default_rng(16)
    Hkv = 3
    prior = [0, 1, P - 1, P, P + 1, 3 * P - 2]
    n_new = [1, P, 2, 1, 2 * P + 3, 5]
    T = len(prior)
    pages = [(a + b + P - 1) // P for a, b in zip(prior, n_new)]
    num_pages = sum(pages) + 4
    perm = rng.permutation(num_pages)
    table = np.full((T, max(pages) + 2), -1, np.int32)
    o = 0
    for t in range(T):
        table[t, :pages[t]] = perm[o:o + pages[t]]
        o += pages[t]
    k_pool = rng.integers(0, 65536, size=(num_pages, Hkv, P, D), dtype=np.uint16)
    v_pool = rng.integers(0, 65536, size=(num_pages, Hkv, P, D), dtype=np.uint16)
    k0, v0 = k_pool.copy(), v_pool.copy()
    indptr = np.concatenate([[0], np.cumsum(n_new)]).astype(np.int32)
    k_new = rng.integers(0, 65536, size=(int(indptr[-1]), Hkv, D), dtype=np.uint16)
    v_new = rng.integers(0, 65536, size=(int(indptr[-1]), Hkv, D), dtype=np.uint16)
    after = oracle.kv_append(k_pool, v_pool, table, np.array(prior, np.int32), indptr, k_new, v_new)
    assert list(after) == [a + b for a, b in zip(prior, n_new)]
    touched = np.zeros((num_pages, P), bool)
    for t in range(T):
        for r in range(n_new[t]):
            pos = prior[t] + r
            pg, sl = table[t, pos // P], pos % P
            assert not touched[pg, sl]
            touched[pg, sl] = True
            assert np.array_equal(k_pool[pg, :, sl, :], k_new[indptr[t] + r])
            assert np.array_equal(v_pool[pg, :, sl, :], v_new[indptr[t] + r])
    keep = np.broadcast_to(~touched[:, None, :, None], k_pool.shape)
    assert np.array_equal(k_pool[keep], k0[keep]) and np.array_equal(v_pool[keep], v0[keep])
    assert touched.sum() == indptr[-1]


def test_append_with_traj_ids_and_errors():
    rng = np.random.default_rng(17)
    P, Hkv = 16, 1
    table = np.array([[0, 1], [2, 3], [4, -1]], np.int32)
    k_pool = np.zeros((5, Hkv, P, D), np.uint16)
    v_pool = np.zeros((5, Hkv, P, D), np.uint16)
    lens = np.array([3, 16, 10], np.int32)
    k_new = rng.integers(1, 65536, size=(3, Hkv, D), dtype=np.uint16)
    v_new = rng.integers(1, 65536, size=(3, Hkv, D), dtype=np.uint16)
    after = oracle.kv_append(k_pool, v_pool, table, lens, np.array([0, 2, 3], np.int32), k_new, v_new,
                             traj_ids=np.array([1, 0], np.int32))
    assert list(after) == [4, 18, 10]
    assert np.array_equal(k_pool[3, 0, 0], k_new[0, 0]) and np.array_equal(k_pool[3, 0, 1], k_new[1, 0])
    assert np.array_equal(v_pool[0, 0, 3], v_new[2, 0])
    assert k_pool[4].sum() == 0
    # growing trajectory 2 past the page it owns hits the -1 entry
    with pytest.raises(oracle.OracleError):
        oracle.kv_append(k_pool, v_pool, table, lens, np.array([0, 7], np.int32),
                         np.zeros((7, Hkv, D), np.uint16), np.zeros((7, Hkv, D), np.uint16),
                         traj_ids=np.array([2], np.int32))


# ---- P15: brute force on tiny inputs, independent scalar routine in extended precision --------------
def test_brute_force_tiny():
    rng = np.random.default_rng(18)
    Dt, Hq, Hkv, P = 4, 4, 2, 2
    g = Hq // Hkv
    for trial in range(40):
        L = int(rng.integers(1, 9))
        Kf = rng.integers(-1, 2, size=(L, Hkv, Dt)).astype(np.float32)
        Vf = rng.integers(-1, 2, size=(L, Hkv, Dt)).astype(np.float32)
        qf = rng.integers(-1, 2, size=(1, Hq, Dt)).astype(np.float32)
        kp, vp, table, lens = pack_pages([to_bf16_bits(Kf)], [to_bf16_bits(Vf)], P, Hkv, Dt, rng=rng)
        out, lse = oracle.decode_attn(kp, vp, table, lens, to_bf16_bits(qf), 0.75)
        for hq in range(Hq):
            h = hq // g
            s = [np.longdouble(0.75) * sum(np.longdouble(qf[0, hq, d]) * np.longdouble(Kf[j, h, d]) for d in range(Dt))
                 for j in range(L)]
            Z = sum(np.exp(sj) for sj in s)
            for d in range(Dt):
                ref = sum(np.exp(s[j]) * np.longdouble(Vf[j, h, d]) for j in range(L)) / Z
                assert abs(float(ref) - out[0, hq, d]) < 1e-14
            assert abs(float(np.log(Z)) - lse[0, hq]) < 1e-14


# ---- P16: poison immunity ------------------------------------------------------------------------
@pytest.mark.parametrize("bits", [0x7FC0, 0x7F80, 0xFF80, 0x7F7F])
def test_dead_slots_and_table_tail_do_not_matter(bits):
    rng = np.random.default_rng(19)
    K, V, q = make_case(rng, [5, 16, 35], 4, 2)
    ref = run_decode(K, V, q, 0.1, 16, fill_bits=0)
    got = run_decode(K, V, q, 0.1, 16, rng=np.random.default_rng(5), fill_bits=bits, spare=9,
                     table_fill=10 ** 6, max_pages=7)
    assert np.array_equal(ref[0], got[0]) and np.array_equal(ref[1], got[1])
    assert np.all(np.isfinite(got[0]))


def test_shared_prefix_pages_may_alias():
    rng = np.random.default_rng(20)
    K, V, q = make_case(rng, [32 + 7], 2, 1)
    kp, vp, table, lens = pack_pages(K, V, 16, 1, D, spare=4)
    # second trajectory shares the two full prefix pages and owns a different tail page
    tail2 = rand_bits(rng, 3, 1, D)
    kp[4, 0, :3] = tail2[:, 0]
    vp[4, 0, :3] = tail2[:, 0]
    table2 = np.array([table[0], [table[0, 0], table[0, 1], 4]], np.int32)
    q2 = np.concatenate([q, q])
    out, _ = oracle.decode_attn(kp, vp, table2, np.array([39, 35], np.int32), q2, 0.1)
    K_b = np.concatenate([K[0][:32], tail2])
    o_ref, _ = dense_attention(q[0], K_b, K_b * 0 + np.concatenate([V[0][:32], tail2]), 0.1, 2)
    np.testing.assert_allclose(out[1], o_ref, rtol=1e-12, atol=1e-13)


def test_out_of_range_page_is_an_error_not_a_read():
    rng = np.random.default_rng(21)
    K, V, q = make_case(rng, [20], 2, 1)
    kp, vp, table, lens = pack_pages(K, V, 16, 1, D)
    bad = table.copy()
    bad[0, 1] = kp.shape[0]
    with pytest.raises(oracle.OracleError):
        oracle.decode_attn(kp, vp, bad, lens, q, 1.0)
    with pytest.raises(oracle.OracleError):
        oracle.decode_attn(kp, vp, table, np.array([33], np.int32), q, 1.0)   # longer than the table row


# ---- gather: the inverse of append ---------------------------------------------------------------
@pytest.mark.parametrize("P", [16, 64])
def test_gather_returns_what_was_packed_and_inverts_append(P):
    rng = np.random.default_rng(30)
    lens = [1, P - 1, P, P + 1, 3 * P + 5]
    K = [rng.integers(0, 65536, size=(L, 2, D), dtype=np.uint16) for L in lens]
    V = [rng.integers(0, 65536, size=(L, 2, D), dtype=np.uint16) for L in lens]
    kp, vp, table, sl = pack_pages(K, V, P, 2, D, rng=rng, fill_bits=0xFFFF)
    indptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ko, vo = oracle.kv_gather(kp, vp, table, sl, indptr)
    assert np.array_equal(ko, np.concatenate(K)) and np.array_equal(vo, np.concatenate(V))
    # a subset, in another order, and only a prefix of one trajectory
    ids = np.array([4, 1], np.int32)
    ko2, vo2 = oracle.kv_gather(kp, vp, table, sl, np.array([0, 2 * P + 1, 2 * P + 1 + lens[1]], np.int32), traj_ids=ids)
    assert np.array_equal(ko2, np.concatenate([K[4][:2 * P + 1], K[1]]))
    # gather then append into an empty pool with a different page table reproduces the logical contents
    kp2 = np.zeros_like(kp); vp2 = np.zeros_like(vp)
    table2 = table[:, ::-1].copy() if False else np.where(table >= 0, kp.shape[0] - 1 - table, -1).astype(np.int32)
    after = oracle.kv_append(kp2, vp2, table2, np.zeros(len(lens), np.int32), indptr, ko, vo)
    assert list(after) == lens
    ko3, vo3 = oracle.kv_gather(kp2, vp2, table2, after, indptr)
    assert np.array_equal(ko3, ko) and np.array_equal(vo3, vo)
    with pytest.raises(oracle.OracleError):      # asking for more rows than the trajectory holds
        oracle.kv_gather(kp, vp, table, sl, np.array([0, lens[0] + 1], np.int32))
