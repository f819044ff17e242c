"""Pins for the oracle's E4M3 code (fp8 KV pools): the published format's closed forms, exhaustive round trips,
tie and saturation cases, and the fp8 attention path against the bf16 one on exactly representable data."""
import math

import numpy as np
import pytest

import oracle


def test_decode_matches_the_format_definition_for_every_code():
    # E4M3: value = (-1)^s * 2^(e-7) * (1 + m/8) for e in 1..15, 2^-6 * m/8 for e = 0; S.1111.111 is NaN
    codes = np.arange(256, dtype=np.uint8)
    got = oracle.e4m3_decode(codes)
    for c in range(256):
        s, e, m = c >> 7, (c >> 3) & 15, c & 7
        if e == 15 and m == 7:
            assert math.isnan(got[c])
            continue
        want = (m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7)
        assert got[c] == (-want if s else want), c
    assert got[0x7E] == 448.0 and got[0x01] == 2.0 ** -9 and got[0x38] == 1.0 and got[0xC0] == -2.0


def test_encode_round_trips_every_finite_code_and_is_monotone():
    codes = np.arange(256, dtype=np.uint8)
    vals = oracle.e4m3_decode(codes)
    fin = ~np.isnan(vals)
    assert np.array_equal(oracle.e4m3_encode(vals[fin].astype(np.float32)), codes[fin])
    xs = np.linspace(-500, 500, 200001).astype(np.float32)
    dec = oracle.e4m3_decode(oracle.e4m3_encode(xs))
    assert np.all(np.diff(dec) >= 0)
    # nearest: the error never exceeds half the gap to the neighbouring codes
    pos = np.sort(vals[fin & (vals >= 0)])
    inside = np.abs(xs) <= 448
    idx = np.clip(np.searchsorted(pos, np.abs(xs[inside])), 1, len(pos) - 1)
    gap = pos[idx] - pos[idx - 1]
    assert np.all(np.abs(np.abs(dec[inside]) - np.abs(xs[inside].astype(np.float64))) <= gap / 2 + 1e-12)


def test_ties_go_to_the_even_code_and_large_values_saturate():
    pos = np.sort(oracle.e4m3_decode(np.arange(0x7F, dtype=np.uint8)))       # 0 .. 448
    mids = ((pos[:-1] + pos[1:]) / 2).astype(np.float32)                      # exactly representable in fp32
    got = oracle.e4m3_encode(mids)
    lo = oracle.e4m3_encode(pos[:-1].astype(np.float32))
    for k in range(len(mids)):
        even = lo[k] if lo[k] % 2 == 0 else lo[k] + 1
        assert got[k] == even, (k, mids[k])
    eps = np.float32(1.0 + 2.0 ** -20)
    assert np.array_equal(oracle.e4m3_encode(mids[1:] * eps), lo[1:] + 1)     # just above a midpoint: up
    assert np.array_equal(oracle.e4m3_encode(mids[1:] / eps), lo[1:])         # just below: down
    big = np.array([448, 449, 464, 480, 1e9, np.inf, -449, -np.inf], np.float32)
    assert list(oracle.e4m3_encode(big)) == [0x7E] * 6 + [0xFE] * 2
    assert oracle.e4m3_encode(np.array([np.nan], np.float32))[0] == 0x7F
    assert list(oracle.e4m3_encode(np.array([0.0, -0.0, 2.0 ** -10, 2.0 ** -10 * 1.001], np.float32))) == [0, 0x80, 0, 1]


def test_quantised_append_is_encode_of_scaled_rows_in_fp32_then_a_bit_copy():
    rng = np.random.default_rng(0)
    P, H, D = 16, 2, 128
    table = np.array([[3, 1], [0, 2]], np.int32)
    lens = np.array([5, 14], np.int32)
    indptr = np.array([0, 4, 7], np.int32)
    rows = (rng.standard_normal((7, H, D)) * 3).astype(np.float32)
    bits = (rows.view(np.uint32) >> 16).astype(np.uint16)                     # bf16 by truncation: any bf16 will do
    k8 = np.full((4, H, P, D), 0x55, np.uint8)
    v8 = np.full((4, H, P, D), 0xAA, np.uint8)
    after = oracle.kv_append_fp8(k8, v8, table, lens, indptr, bits, bits, 0.05, 0.2)
    assert list(after) == [9, 17]
    x = (bits.astype(np.uint32) << 16).view(np.float32)
    kq = oracle.e4m3_encode(x * (np.float32(1) / np.float32(0.05)))
    vq = oracle.e4m3_encode(x * (np.float32(1) / np.float32(0.2)))
    touched = np.zeros((4, P), bool)
    for i, t in enumerate([0, 1]):
        for r in range(indptr[i + 1] - indptr[i]):
            pos = lens[t] + r
            pg = table[t, pos // P]
            assert np.array_equal(k8[pg, :, pos % P], kq[indptr[i] + r])
            assert np.array_equal(v8[pg, :, pos % P], vq[indptr[i] + r])
            touched[pg, pos % P] = True
    assert np.all(k8[~touched[:, None, :].repeat(H, 1)] == 0x55) and np.all(v8[~touched[:, None, :].repeat(H, 1)] == 0xAA)


def test_fp8_attention_equals_bf16_attention_on_the_dequantised_pool():
    # every finite code value is a bf16 value: decoding over the codes with scales (ks, vs) must equal bf16 decoding
    # over the values with sm_scale * ks, times vs
    rng = np.random.default_rng(1)
    P, H, D, L = 16, 2, 128, 70
    codes_k = rng.integers(0, 256, (5, H, P, D)).astype(np.uint8)
    codes_v = rng.integers(0, 256, (5, H, P, D)).astype(np.uint8)
    codes_k[(codes_k & 0x7F) == 0x7F] = 0x10                                  # no NaN codes among the live data
    codes_v[(codes_v & 0x7F) == 0x7F] = 0x10
    codes_k = (codes_k & 0x80) | np.minimum(codes_k & 0x7F, 0x3F)            # |value| < 2: moderate scores
    table = np.array([[4, 2, 0, 1, 3]], np.int32)
    lens = np.array([L], np.int32)
    q = ((rng.standard_normal((1, 4, D)) * 0.5).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    out, lse = oracle.decode_attn_fp8(codes_k, codes_v, table, lens, q, 0.25, 0.5, 2.0)
    kv = oracle.e4m3_decode(codes_k)[table[0]].transpose(1, 0, 2, 3).reshape(H, -1, D)[:, :L]
    vv = oracle.e4m3_decode(codes_v)[table[0]].transpose(1, 0, 2, 3).reshape(H, -1, D)[:, :L]
    qf = (q.astype(np.uint32) << 16).view(np.float32).astype(np.float64)[0]
    for hq in range(4):
        h = hq // 2
        s = 0.25 * 0.5 * (kv[h] @ qf[hq])
        w = np.exp(s - s.max())
        np.testing.assert_allclose(out[0, hq], 2.0 * (w @ vv[h]) / w.sum(), rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(lse[0, hq], s.max() + math.log(w.sum()), rtol=1e-12)


def test_hand_over_of_codes_is_a_bit_copy_token_by_token():
    # gather then append onto another pool with another page table: every live token's codes arrive unchanged, in
    # order; checked with plain loops over (trajectory, position)
    rng = np.random.default_rng(2)
    P, H, D = 16, 3, 128
    src_k = rng.integers(0, 256, (7, H, P, D)).astype(np.uint8)
    src_v = rng.integers(0, 256, (7, H, P, D)).astype(np.uint8)
    table = np.array([[5, 0, 3], [6, 2, -1], [1, 4, -1]], np.int32)
    lens = np.array([40, 17, 0], np.int32)
    ids = np.array([1, 0], np.int32)                                          # hand over trajectory 1, then 0
    n = np.array([17, 33], np.int32)                                          # all of 1, the first 33 tokens of 0
    indptr = np.array([0, 17, 50], np.int32)
    gk, gv = oracle.kv_gather_fp8(src_k, src_v, table, lens, indptr, traj_ids=ids)
    assert gk.shape == (50, H, D) and gk.dtype == np.uint8
    for i, t in enumerate(ids):
        for pos in range(n[i]):
            assert np.array_equal(gk[indptr[i] + pos], src_k[table[t, pos // P], :, pos % P])
            assert np.array_equal(gv[indptr[i] + pos], src_v[table[t, pos // P], :, pos % P])
    dst_k = np.full((6, H, P, D), 0x55, np.uint8)
    dst_v = np.full((6, H, P, D), 0xAA, np.uint8)
    dtable = np.array([[2, 0, 4], [1, 5, 3]], np.int32)
    dlens = np.array([3, 0], np.int32)                                        # receiver 0 already holds 3 tokens
    after = oracle.kv_append_fp8_codes(dst_k, dst_v, dtable, dlens, indptr, gk, gv)
    assert list(after) == [20, 33]
    touched = np.zeros((6, P), bool)
    for i in range(2):
        for r in range(n[i]):
            pos = dlens[i] + r
            pg = dtable[i, pos // P]
            assert np.array_equal(dst_k[pg, :, pos % P], gk[indptr[i] + r]) and np.array_equal(dst_v[pg, :, pos % P], gv[indptr[i] + r])
            touched[pg, pos % P] = True
    assert np.all(dst_k[~touched[:, None, :].repeat(H, 1)] == 0x55) and np.all(dst_v[~touched[:, None, :].repeat(H, 1)] == 0xAA)


def test_fp8_chunk_rows_against_a_dense_evaluation_and_against_decode():
    # chunk row j of n sees the first L - n + j + 1 keys: each row checked against numpy over the dequantised
    # context, and the last row against the fp8 decode call (which sees all L keys)
    rng = np.random.default_rng(3)
    P, H, D = 16, 2, 128
    codes_k = rng.integers(0, 256, (6, H, P, D)).astype(np.uint8)
    codes_v = rng.integers(0, 256, (6, H, P, D)).astype(np.uint8)
    codes_k = (codes_k & 0x80) | np.minimum(codes_k & 0x7F, 0x3F)            # |value| < 2: moderate scores, no NaN
    codes_v[(codes_v & 0x7F) == 0x7F] = 0x10
    table = np.array([[4, 2, 0, 5], [1, 3, -1, -1]], np.int32)
    lens = np.array([55, 20], np.int32)
    n = [9, 20]                                                               # trajectory 1: the whole context is the chunk
    q_indptr = np.array([0, 9, 29], np.int32)
    q = ((rng.standard_normal((29, 4, D)) * 0.5).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    ks, vs, sm = 0.5, 2.0, 0.25
    out, lse = oracle.obs_chunk_attn_fp8(codes_k, codes_v, table, lens, q_indptr, q, sm, ks, vs)
    assert out.shape == (29, 4, D) and lse.shape == (29, 4)
    qf = (q.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for t in range(2):
        npg = (lens[t] + P - 1) // P
        kv = oracle.e4m3_decode(codes_k)[table[t, :npg]].transpose(1, 0, 2, 3).reshape(H, -1, D)
        vv = oracle.e4m3_decode(codes_v)[table[t, :npg]].transpose(1, 0, 2, 3).reshape(H, -1, D)
        for j in range(n[t]):
            c = lens[t] - n[t] + j + 1
            r = q_indptr[t] + j
            for hq in range(4):
                s = sm * ks * (kv[hq // 2, :c] @ qf[r, hq])
                w = np.exp(s - s.max())
                np.testing.assert_allclose(out[r, hq], vs * (w @ vv[hq // 2, :c]) / w.sum(), rtol=1e-12, atol=1e-12)
                np.testing.assert_allclose(lse[r, hq], s.max() + math.log(w.sum()), rtol=1e-12)
    last = q_indptr[1:] - 1
    d_out, d_lse = oracle.decode_attn_fp8(codes_k, codes_v, table, lens, q[last], sm, ks, vs)
    np.testing.assert_allclose(out[last], d_out, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(lse[last], d_lse, rtol=1e-13)
