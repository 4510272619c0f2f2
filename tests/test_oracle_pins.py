"""Pins for the CPU checker: each function is held against something it did not
compute itself -- values the paper prints, closed forms, brute force on tiny
inputs, textbook attention from a library, and invariants the paper states."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
SCALE = 1.0 / math.sqrt(128.0)


def bf16(x: torch.Tensor) -> np.ndarray:
    return O.bf16_bits(x.to(torch.bfloat16))


def f32(bits: np.ndarray) -> np.ndarray:
    return O.bits_to_f32(bits)


def rng(seed):
    g = torch.Generator()
    g.manual_seed(seed)
    return g


# --------------------------------------------------------------------- metadata
def test_page_meta_is_min_max_of_valid_tokens():
    g = rng(1)
    T = 16 * 5 + 7                      # ragged last page
    k = bf16(torch.randn(T, 128, generator=g))
    kmin, kmax = O.page_meta(k, T)
    kf = f32(k)
    assert kmin.shape == (6, 128)
    for p in range(6):
        rows = kf[p * 16:min(T, (p + 1) * 16)]
        np.testing.assert_array_equal(f32(kmin[p]), rows.min(0))
        np.testing.assert_array_equal(f32(kmax[p]), rows.max(0))
    # containment: every key lies between its page's bounds
    pid = np.arange(T) // 16
    assert (f32(kmin)[pid] <= kf).all() and (kf <= f32(kmax)[pid]).all()


def test_page_meta_respects_length_and_zero_signs():
    k = np.zeros((32, 128), np.uint16)
    k[0, :] = 0x8000                    # -0.0
    k[1, :] = 0x0000                    # +0.0
    k[20:, :] = 0x7F00                  # huge values past the valid length
    kmin, kmax = O.page_meta(k, 18)
    assert kmin.shape[0] == 2
    assert (kmin[0] == 0x8000).all() and (kmax[0] == 0x0000).all()   # -0 orders below +0
    assert (kmax[1] == 0).all()         # tokens 16,17 only; tokens >= 18 ignored


# ------------------------------------------------------------------ page bound
def test_bound_dominates_every_token_logit():
    g = rng(2)
    T = 16 * 8
    k = bf16(torch.randn(T, 128, generator=g) * 3)
    kmin, kmax = O.page_meta(k, T)
    for trial in range(4):
        q = bf16(torch.randn(128, generator=g))
        logits = f32(k).astype(np.float64) @ f32(q).astype(np.float64)
        for p in range(8):
            u = O.bound_f32(q, kmin[p], kmax[p])
            tol = 128 * 2.0 ** -24 * np.abs(f32(q).astype(np.float64) * f32(kmax[p])).sum()
            assert u + tol >= logits[p * 16:(p + 1) * 16].max()


def test_bound_of_single_token_page_is_the_dot_product():
    g = rng(3)
    q = bf16(torch.randn(128, generator=g))
    k = bf16(torch.randn(1, 128, generator=g))
    kmin, kmax = O.page_meta(k, 1)
    exact = float(f32(q).astype(np.float64) @ f32(k[0]).astype(np.float64))
    assert O.bound_f64(q, kmin[0], kmax[0]) == pytest.approx(exact, abs=1e-12)
    err = 128 * 2.0 ** -24 * float(np.abs(f32(q).astype(np.float64) * f32(k[0])).sum())
    assert abs(O.bound_f32(q, kmin[0], kmax[0]) - exact) <= err


def test_bound_negative_query_uses_the_minimum():
    # one channel, q = -2, keys in [3, 5]: max(q*3, q*5) = -6
    q = bf16(torch.zeros(128)); kmin = q.copy(); kmax = q.copy()
    q[7] = bf16(torch.tensor([-2.0]))[0]
    kmin[7] = bf16(torch.tensor([3.0]))[0]
    kmax[7] = bf16(torch.tensor([5.0]))[0]
    assert O.bound_f32(q, kmin, kmax) == -6.0
    assert O.bound_f64(q, kmin, kmax) == -6.0


def _bound_with_terms(terms):
    """Bound of a single-token page whose per-channel term is terms[c] (q = 1)."""
    q = bf16(torch.ones(128))
    k = bf16(torch.tensor(terms, dtype=torch.float32))
    assert (f32(k) == np.asarray(terms, np.float32)).all()
    return O.bound_f32(q, k, k)


def test_bound_summation_order_hand_cases():
    """Hand-worked fp32 results that only the declared order produces."""
    big = float(2 ** 24)
    # (a) partial 0 holds 2^24, partial 1 holds eight ones, partial 8 holds -2^24.
    #     Declared order: distance-8 step cancels the big terms first -> 8.
    #     A left-to-right sum absorbs the ones into 2^24 -> 0.
    t = [0.0] * 128
    t[0] = big
    for c in range(8, 16):
        t[c] = 1.0
    t[64] = -big
    assert _bound_with_terms(t) == 8.0
    # (b) a single one in partial 1: combining at distance 1 first would round
    #     2^24 + 1 to 2^24 and lose it; the declared order (8 first) keeps it.
    t = [0.0] * 128
    t[0] = big; t[8] = 1.0; t[64] = -big
    assert _bound_with_terms(t) == 1.0
    # (c) inside a partial, even and odd channels are summed separately:
    #     even = 2^24 - 2^24 = 0, odd = 1, partial = 1 (one running sum over all
    #     eight channels would round 2^24 + 1 to 2^24 and give 0).
    t = [0.0] * 128
    t[0] = big; t[1] = 1.0; t[2] = -big
    assert _bound_with_terms(t) == 1.0
    # (d) each of the two running sums goes left to right: (2^24 + 1) rounds to
    #     2^24 before -2^24 arrives, so the one is lost, on the even side ...
    t = [0.0] * 128
    t[0] = big; t[2] = 1.0; t[4] = -big
    assert _bound_with_terms(t) == 0.0
    #     ... and on the odd side.
    t = [0.0] * 128
    t[1] = big; t[3] = 1.0; t[7] = -big
    assert _bound_with_terms(t) == 0.0
    # (e) partials are 8 channels wide: channel 8 starts a new partial, so the
    #     one survives there.
    t = [0.0] * 128
    t[7] = big; t[8] = 1.0; t[71] = -big
    assert _bound_with_terms(t) == 1.0


def test_page_scores_take_the_max_over_grouped_heads():
    g = rng(4)
    k = bf16(torch.randn(64, 128, generator=g))
    kmin, kmax = O.page_meta(k, 64)
    qg = bf16(torch.randn(7, 128, generator=g))
    u = O.page_scores(qg, kmin, kmax)
    per_head = np.array([[O.bound_f32(qg[h], kmin[p], kmax[p]) for p in range(4)] for h in range(7)])
    np.testing.assert_array_equal(u, per_head.max(0).astype(np.float32))
    # permuting the heads of a group cannot change the scores
    np.testing.assert_array_equal(u, O.page_scores(qg[::-1].copy(), kmin, kmax))


# -------------------------------------------------------------- page selection
def test_select_matches_exhaustive_sort_with_ties():
    g = np.random.default_rng(5)
    for n_pages, budget in [(1, 16), (7, 48), (33, 16 * 9), (64, 16 * 64), (40, 15), (40, 16 * 41)]:
        u = g.integers(-3, 4, n_pages).astype(np.float32)       # many exact ties
        k = min(n_pages, budget // 16)
        order = sorted(range(n_pages), key=lambda p: (-u[p], p))[:k]
        np.testing.assert_array_equal(O.select(u, budget), np.array(sorted(order), np.int32))


def test_select_full_budget_returns_all_pages_and_zero_signs_tie():
    u = np.array([0.0, -0.0, 0.0, -0.0], np.float32)
    np.testing.assert_array_equal(O.select(u, 64), [0, 1, 2, 3])
    np.testing.assert_array_equal(O.select(u, 32), [0, 1])       # -0 == +0: lower id wins
    np.testing.assert_array_equal(O.select(np.array([1, 5, 5, 2], np.float32), 32), [1, 2])


# --------------------------------------------------------------------- routing
def popcount(m):
    return np.array([bin(int(x)).count("1") for x in np.asarray(m).ravel()]).reshape(np.shape(m))


def test_route_global_budget_invariants():
    g = np.random.default_rng(6)
    for S, K in [(8, 4), (16, 4), (8, 1), (8, 8), (4, 1), (16, 14)]:
        N = 257
        sc = g.standard_normal((N, S)).astype(np.float32)
        rc, mask = O.route(sc, None, S, K, min_per_token=1)
        assert rc == 0
        cnt = popcount(mask)
        assert cnt.sum() == N * K                       # M = N*K (Appendix B.1)
        assert cnt.min() >= 1 and cnt.max() <= S
        if K == S:
            assert (mask == (1 << S) - 1).all()
        if K == 1:
            np.testing.assert_array_equal(mask, (1 << sc.argmax(1)).astype(np.uint16))
        # every kept pair that is not a token's reserved best scores at least as
        # high as every dropped pair
        bits = (mask[:, None] >> np.arange(S)) & 1
        reserved = np.zeros_like(bits); reserved[np.arange(N), sc.argmax(1)] = 1
        kept_free = sc[(bits == 1) & (reserved == 0)]
        dropped = sc[bits == 0]
        if kept_free.size and dropped.size:
            assert kept_free.min() >= dropped.max()


def test_route_global_without_floor_reproduces_fig1_properties():
    # Fig. 1: S = 4, average budget 1.0, K_j ranges over {0..S} with some tokens at 0.
    g = np.random.default_rng(7)
    N, S = 4096, 4
    # token-level relevance shifts all of a token's logits together, as in the figure
    sc = (g.standard_normal((N, 1)) * 2 + g.standard_normal((N, S))).astype(np.float32)
    rc, mask = O.route(sc, None, S, 1, min_per_token=0)
    cnt = popcount(mask)
    assert rc == 0 and cnt.sum() == N                   # mean allocation = 1.0
    assert cnt.min() == 0 and cnt.max() == S
    # exactly the N highest-scoring pairs
    thr = np.sort(sc.ravel())[::-1][N - 1]
    bits = (mask[:, None] >> np.arange(S)) & 1
    assert ((sc > thr) <= (bits == 1)).all() and ((bits == 1) <= (sc >= thr)).all()


def test_route_floor_equals_best_feasible_subset_by_enumeration():
    g = np.random.default_rng(8)
    S = 4
    for N, K in [(2, 1), (3, 2), (4, 2), (3, 3), (4, 1)]:
        sc = g.permutation(N * S).astype(np.float32).reshape(N, S)     # distinct scores
        rc, mask = O.route(sc, None, S, K, min_per_token=1)
        best, best_sets = -np.inf, None
        for sub in itertools.combinations(range(N * S), N * K):
            m = np.zeros(N * S, bool); m[list(sub)] = True
            if not m.reshape(N, S).any(1).all():
                continue
            val = sc.ravel()[m].sum()
            if val > best:
                best, best_sets = val, m.reshape(N, S)
        got = ((mask[:, None] >> np.arange(S)) & 1).astype(bool)
        assert rc == 0
        np.testing.assert_array_equal(got, best_sets)


def test_route_ties_go_to_lower_flat_index_and_classes():
    S = 4
    sc = np.zeros((6, S), np.float32)                    # everything ties
    cls = np.array([1, 2, 0, 1, 1, 1], np.uint8)         # routed, full, drop, routed x3
    rc, mask = O.route(sc, cls, S, 2, min_per_token=1)
    # N = 4 routed tokens, M = 8: reserve group 0 of each, then the 4 lowest flat
    # indices among the rest: token 0 groups 1,2,3 and token 3 group 1.
    assert rc == 0
    np.testing.assert_array_equal(mask, [0b1111, 0b1111, 0, 0b0011, 0b0001, 0b0001])
    rc, _ = O.route(sc, cls, S, 0, min_per_token=1)
    assert rc == -1                                       # budget below one group per token
    rc, mask = O.route(sc, cls, S, 0, min_per_token=0)
    assert rc == 0 and list(mask) == [0, 0b1111, 0, 0, 0, 0]


def test_route_per_token_topk():
    g = np.random.default_rng(9)
    for S, K in [(4, 1), (8, 2), (16, 4)]:               # the paper's VLM grid (Appendix C.2)
        sc = g.standard_normal((100, S)).astype(np.float32)
        rc, mask = O.route(sc, None, S, K, mode=O.MODE_PER_TOKEN)
        top = np.argsort(-sc, axis=1, kind="stable")[:, :K]
        want = np.zeros(100, np.uint16)
        for j in range(K):
            want |= (1 << top[:, j]).astype(np.uint16)
        assert rc == 0
        np.testing.assert_array_equal(mask, want)


# --------------------------------------------------------------------- packing
def test_pack_roundtrip_and_offsets():
    g = rng(10)
    T, S = 100, 8
    v = bf16(torch.randn(T, 128, generator=g))
    mask = np.random.default_rng(10).integers(0, 1 << S, T).astype(np.uint16)
    mask[3] = 0; mask[4] = (1 << S) - 1
    total, offs, packed = O.pack(v, mask, S, 1000)
    cnt = popcount(mask)
    assert total == cnt.sum() == offs[T]
    np.testing.assert_array_equal(np.diff(offs.astype(np.int64)), cnt)
    dense = np.zeros_like(v)
    for t in range(T):
        slot = offs[t]
        for j in range(S):
            if (mask[t] >> j) & 1:
                dense[t, j * 16:(j + 1) * 16] = packed[slot]; slot += 1
    keep = np.repeat((mask[:, None] >> np.arange(S)) & 1, 16, axis=1).astype(bool)
    np.testing.assert_array_equal(dense, np.where(keep, v, 0))
    over, _, _ = O.pack(v, mask, S, int(total) - 1)
    assert over == -1


def test_stored_bytes_reproduce_the_printed_kv_fractions():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "kv_fractions.txt")) if l[0].isdigit()]
    assert len(rows) == 14
    g = np.random.default_rng(11)
    for r, K, S, pct, *_ in rows:
        r, K, S, pct = float(r), int(K), int(S), float(pct)
        T0 = 2048
        N = int(T0 * r)
        sc = g.standard_normal((N, S)).astype(np.float32)
        rc, mask = O.route(sc, None, S, K, min_per_token=1)
        v = np.zeros((N, 128), np.uint16)
        total, _, _ = O.pack(v, mask, S, N * S)
        frac = O.kv_fraction(T0, N, total, S)
        assert frac == r * (1 + K / S) / 2                # exact in binary
        assert round(100 * frac + 1e-9, 3) == pytest.approx(pct, abs=5.1e-4)
    assert O.kv_fraction(2048, 512, 512 * 2, 8) == 0.15625
    assert O.kv_fraction(2048, 256, 256 * 2, 8) == 0.078125


# ------------------------------------------------------------------- attention
def _setup_attn(seed, T, S, K):
    g = rng(seed)
    q = bf16(torch.randn(128, generator=g))
    k = bf16(torch.randn(T, 128, generator=g))
    v = bf16(torch.randn(T, 128, generator=g))
    sc = torch.randn(T, S, generator=g).numpy()
    rc, mask = O.route(sc, None, S, K, min_per_token=1)
    total, offs, packed = O.pack(v, mask, S, T * S)
    return q, k, v, mask, offs, packed


def _dense_reference(q, k, v_eff):
    """Textbook softmax attention in fp64 through torch's library routine."""
    qt = torch.from_numpy(f32(q).astype(np.float64))[None, None, None, :]
    kt = torch.from_numpy(f32(k).astype(np.float64))[None, None]
    vt = torch.from_numpy(v_eff.astype(np.float64))[None, None]
    return torch.nn.functional.scaled_dot_product_attention(qt, kt, vt)[0, 0, 0].numpy()


def test_attend_all_groups_equals_dense_softmax_attention():
    T, S = 16 * 6 + 5, 8
    q, k, v, mask, offs, packed = _setup_attn(12, T, S, S)
    assert (mask == 0xFF).all()
    out, lse = O.attend_packed(q, k, packed, mask, offs, T, S, None, SCALE)
    np.testing.assert_allclose(out, _dense_reference(q, k, f32(v)), rtol=0, atol=1e-12)
    s = (f32(k).astype(np.float64) @ f32(q).astype(np.float64)) * SCALE
    assert lse == pytest.approx(float(np.log(np.exp(s - s.max()).sum()) + s.max()), abs=1e-12)


def test_attend_masked_equals_dense_attention_over_zero_filled_values():
    for S, K in [(8, 4), (16, 4), (4, 1)]:
        T = 16 * 9 + 3
        q, k, v, mask, offs, packed = _setup_attn(13 + S, T, S, K)
        keep = np.repeat((mask[:, None] >> np.arange(S)) & 1, 128 // S, axis=1)
        want = _dense_reference(q, k, f32(v) * keep)     # normaliser over every token
        out_p, lse_p = O.attend_packed(q, k, packed, mask, offs, T, S, None, SCALE)
        out_d, lse_d = O.attend_masked_dense(q, k, v, mask, T, S, None, SCALE)
        np.testing.assert_allclose(out_p, want, rtol=0, atol=1e-12)
        np.testing.assert_array_equal(out_p, out_d)      # packed store == masked dense, bit for bit
        assert lse_p == lse_d


def test_attend_zero_group_tokens_still_normalise():
    # two tokens with equal logits; the second keeps no group: out = v0 / 2, not v0
    S = 4
    q = bf16(torch.zeros(128))
    k = bf16(torch.zeros(2, 128))
    v = bf16(torch.ones(2, 128))
    mask = np.array([0b1111, 0], np.uint16)
    total, offs, packed = O.pack(v, mask, S, 8)
    out, lse = O.attend_packed(q, k, packed, mask, offs, 2, S, None, SCALE)
    np.testing.assert_array_equal(out, np.full(128, 0.5))
    assert lse == pytest.approx(math.log(2.0))


def test_attend_page_subset_order_and_split_merge():
    T, S = 16 * 12 + 9, 8
    q, k, v, mask, offs, packed = _setup_attn(14, T, S, 4)
    ids = np.array([1, 4, 5, 9, 12], np.int32)           # page 12 is the ragged last page
    out, lse = O.attend_packed(q, k, packed, mask, offs, T, S, ids, SCALE)
    tok = np.concatenate([np.arange(p * 16, min(T, p * 16 + 16)) for p in ids])
    keep = np.repeat((mask[:, None] >> np.arange(S)) & 1, 16, axis=1)
    want = _dense_reference(q, k[tok], (f32(v) * keep)[tok])
    np.testing.assert_allclose(out, want, rtol=0, atol=1e-12)
    # order of the list does not matter beyond rounding
    out2, lse2 = O.attend_packed(q, k, packed, mask, offs, T, S, ids[::-1].copy(), SCALE)
    np.testing.assert_allclose(out2, out, rtol=0, atol=1e-13)
    # two halves merged by log-sum-exp reproduce the one-shot result
    oa, la = O.attend_packed(q, k, packed, mask, offs, T, S, ids[:2], SCALE)
    ob, lb = O.attend_packed(q, k, packed, mask, offs, T, S, ids[2:], SCALE)
    m = max(la, lb)
    wa, wb = math.exp(la - m), math.exp(lb - m)
    np.testing.assert_allclose((oa * wa + ob * wb) / (wa + wb), out, rtol=0, atol=1e-13)
    assert m + math.log(wa + wb) == pytest.approx(lse, abs=1e-12)


# ---------------------------------------------------------------------- router
def test_router_logits_one_hot_rows_pick_hidden_channels_and_bias_adds():
    g = rng(20)
    B, T, dm, Hkv, S = 2, 5, 64, 2, 4
    h = bf16(torch.randn(B, T, dm, generator=g))
    w = np.zeros((Hkv * S, dm), np.uint16)
    one = bf16(torch.tensor([1.0]))[0]
    pick = [3, 17, 0, 63, 9, 9, 40, 5]                       # row n copies hidden channel pick[n]
    for n, c in enumerate(pick):
        w[n, c] = one
    out = O.router_logits(h, w, S)
    assert out.shape == (B, Hkv, T, S)
    hf = f32(h).astype(np.float64)
    for n, c in enumerate(pick):
        np.testing.assert_array_equal(out[:, n // S, :, n % S], hf[:, :, c])
    bias = np.arange(B * Hkv * S, dtype=np.float32).reshape(B, Hkv * S) / 4
    out_b = O.router_logits(h, w, S, bias)
    np.testing.assert_array_equal(out_b - out, bias.reshape(B, Hkv, 1, S).astype(np.float64) * np.ones((1, 1, T, 1)))


def test_router_logits_hand_example_and_library_matmul():
    # hand-worked: h = (1, 2, -3, 0.5), two rows of W
    h = bf16(torch.tensor([[[1.0, 2.0, -3.0, 0.5]]]))
    w = bf16(torch.tensor([[2.0, 0.0, 1.0, 4.0], [-1.0, 0.5, 0.0, 2.0]]))
    out = O.router_logits(h, w, 2)
    np.testing.assert_array_equal(out.ravel(), [2 - 3 + 2, -1 + 1 + 1])
    # against the library matmul in fp64 (row n of W, token t -> out[b, n // S, t, n % S])
    g = rng(21)
    B, T, dm, Hkv, S = 2, 37, 96, 3, 8
    hh, ww = bf16(torch.randn(B, T, dm, generator=g)), bf16(torch.randn(Hkv * S, dm, generator=g))
    want = (f32(hh).astype(np.float64) @ f32(ww).astype(np.float64).T).reshape(B, T, Hkv, S).transpose(0, 2, 1, 3)
    np.testing.assert_allclose(O.router_logits(hh, ww, S), want, rtol=0, atol=1e-12)


# --------------------------------------------------------------- batched layer
def test_batched_drivers_agree_with_single_problem_calls():
    from paper_2604_21335_b200 import workload as W
    w = W.shrink(W.get("cfg2"), batch=2, t_cache=16 * 20 + 5, token_budget=16 * 6)
    d = W.make_inputs(w, "cpu")
    seq = np.array([w.t_cache, w.t_cache - 37], np.int32)
    k, v, q = bf16(d["k"]), bf16(d["v"]), bf16(d["q"][0])
    sc = d["scores"].numpy()
    kmin, kmax = O.page_meta_batch(k, seq)
    ids, n, u = O.select_batch(q, kmin, kmax, w.token_budget, w.t_cache, seq, want_scores=True)
    cap = w.t_cache * w.k_nominal
    r = O.route_pack_batch(v, sc, None, w.n_groups, w.k_nominal, cap, seq)
    out, lse = O.attend_batch(q, k, w.n_groups, r["mask"], ids, n, SCALE, packed=r["packed"],
                              offs=r["offs"], seq_len=seq)
    out_d, _ = O.attend_batch(q, k, w.n_groups, r["mask"], ids, n, SCALE, v_dense=v, seq_len=seq)
    np.testing.assert_array_equal(out, out_d)
    for b in range(2):
        L = int(seq[b])
        for hk in range(w.n_kv_heads):
            m1, M1 = O.page_meta(k[b, hk], L)
            P = m1.shape[0]
            np.testing.assert_array_equal(kmin[b, hk, :P], m1)
            qg = q[b, hk * w.gq:(hk + 1) * w.gq]
            u1 = O.page_scores(qg, m1, M1)
            np.testing.assert_array_equal(u[b, hk, :P], u1)
            sel = O.select(u1, w.token_budget)
            np.testing.assert_array_equal(ids[b, hk, :n[b, hk]], sel)
            rc, mk = O.route(sc[b, hk, :L], None, w.n_groups, w.k_nominal)
            np.testing.assert_array_equal(r["mask"][b, hk, :L], mk)
            assert r["total"][b, hk] == L * w.k_nominal and r["status"][b, hk] == 0
            tot, of, pk = O.pack(v[b, hk, :L], mk, w.n_groups, cap)
            np.testing.assert_array_equal(r["offs"][b, hk, :L + 1], of)
            np.testing.assert_array_equal(r["packed"][b, hk, :tot], pk[:tot])
            for j in range(w.gq):
                o1, l1 = O.attend_packed(qg[j], k[b, hk], pk, mk, of, L, w.n_groups, sel, SCALE)
                np.testing.assert_array_equal(out[b, hk * w.gq + j], o1)
                assert lse[b, hk * w.gq + j] == l1


# ---------------------------------------------------------------------- query summary term
def test_query_bias_hand_example_constant_rows_and_empty_region():
    # hand-worked: two query tokens (1, 3) and (3, 5): mean (2, 4); rows (1, -1) -> -2 and (0.5, 0.5) -> 3
    h = bf16(torch.tensor([[[1.0, 3.0], [3.0, 5.0]]]))
    w = bf16(torch.tensor([[1.0, -1.0], [0.5, 0.5]]))
    s_q, bias = O.query_bias(h, w)
    np.testing.assert_array_equal(s_q, [[2.0, 4.0]])
    np.testing.assert_array_equal(bias, [[-2.0, 3.0]])
    # the same rows repeated: the mean is the row itself, one-hot weights pick its channels;
    # a sequence with an empty query region contributes nothing
    g = rng(22)
    row = bf16(torch.randn(3, 1, 32, generator=g))
    hq = np.repeat(row, 7, axis=1)
    wq = np.zeros((4, 32), np.uint16)
    one = bf16(torch.tensor([1.0]))[0]
    for n, c in enumerate([5, 0, 31, 5]):
        wq[n, c] = one
    s_q, bias = O.query_bias(hq, wq, np.array([7, 3, 0], np.int32))
    np.testing.assert_array_equal(s_q[:2], f32(row)[:2, 0].astype(np.float64))
    np.testing.assert_array_equal(bias[:2], f32(row)[:2, 0][:, [5, 0, 31, 5]].astype(np.float64))
    assert not s_q[2].any() and not bias[2].any()


def test_query_bias_is_the_mean_of_the_per_token_logits():
    # linearity: W s_Q = mean_t (W h_t); the per-token logits come from the router pinned above
    g = rng(23)
    B, Lq, dm, Hkv, S = 3, 11, 64, 2, 4
    hq = bf16(torch.randn(B, Lq, dm, generator=g))
    wq = bf16(torch.randn(Hkv * S, dm, generator=g))
    q_len = np.array([11, 4, 1], np.int32)
    s_q, bias = O.query_bias(hq, wq, q_len)
    per_tok = O.router_logits(hq, wq, S)                      # [B, Hkv, Lq, S]
    for b in range(B):
        want = per_tok[b, :, : q_len[b], :].mean(axis=1).reshape(-1)
        np.testing.assert_allclose(bias[b], want, rtol=0, atol=1e-12)
        np.testing.assert_allclose(s_q[b], f32(hq)[b, : q_len[b]].astype(np.float64).mean(axis=0), rtol=0, atol=1e-14)


# ---------------------------------------------------------------------- selection with a recent window
def test_select_recent_window_against_brute_force():
    g = np.random.default_rng(31)
    for n, budget, w in [(40, 160, 4), (40, 160, 0), (40, 160, 10), (40, 160, 25), (7, 1000, 3), (33, 16, 4),
                         (50, 320, 20), (12, 0, 2)]:
        u = g.integers(0, 6, n).astype(np.float32)            # many ties
        ids = O.select(u, budget, w)
        k = min(n, budget // 16)
        ww = min(w, k)
        window = list(range(n - ww, n))
        # exhaustive: rank the pages before the window by (-score, id), take k - ww of them
        rest = sorted(range(n - ww), key=lambda p: (-u[p], p))[: k - ww]
        assert ids.tolist() == sorted(rest + window), (n, budget, w)
        assert len(set(ids.tolist())) == k
    # no window = the plain rule
    u = g.standard_normal(64).astype(np.float32)
    np.testing.assert_array_equal(O.select(u, 256, 0), O.select(u, 256))


def test_pages_to_class_hand_example():
    # two problems, 40-token rows; problem 0 lists pages 2 and 0 of a 35-token sequence (page 2 is partial),
    # problem 1 lists nothing
    ids = np.array([[[2, 0, 1], [1, 1, 1]]], np.int32)
    n = np.array([[2, 0]], np.int32)
    cls = O.pages_to_class(ids, n, 40, np.array([35], np.int32))
    want0 = np.zeros(40, np.uint8); want0[0:16] = 1; want0[32:35] = 1
    assert cls.shape == (1, 2, 40)
    np.testing.assert_array_equal(cls[0, 0], want0)
    assert (cls[0, 1] == 0).all()


def test_near_tie_count_on_a_constructed_row_of_bounds():
    # One channel carries the whole bound: q[0] = 1, kmin[p][0] = kmax[p][0] = value_p, so U[p] = value_p exactly
    # (values are exact in bf16).  k = 3 pages: sorted values 9, 8, [5], 5, 5, 4.984375(bf16 step 2^-6 below 5), 1.
    bf = lambda x: (np.array([x], np.float32).view(np.uint32) >> 16).astype(np.uint16)[0]
    vals = [5.0, 9.0, 1.0, 5.0, 8.0, 4.96875, 5.0]
    P_ = len(vals)
    kmin = np.zeros((1, 1, P_, 128), np.uint16); kmax = np.zeros((1, 1, P_, 128), np.uint16)
    for p, x in enumerate(vals):
        assert np.float32(x) == O.bits_to_f32(np.array([bf(x)], np.uint16))[0]
        kmin[0, 0, p, 0] = kmax[0, 0, p, 0] = bf(x)
    q = np.zeros((1, 1, 128), np.uint16); q[0, 0, 0] = bf(1.0)
    T = 16 * P_
    assert O.near_ties_batch(q, kmin, kmax, 3 * 16, T)[0, 0] == 2            # the two other pages equal to 5
    assert O.near_ties_batch(q, kmin, kmax, 3 * 16, T, rel=0.01)[0, 0] == 3  # 4.96875 is within 1 % of 5
    assert O.near_ties_batch(q, kmin, kmax, 1 * 16, T)[0, 0] == 0            # 9 stands alone
    assert O.near_ties_batch(q, kmin, kmax, 2 * 16, T)[0, 0] == 0            # so does 8
    assert O.near_ties_batch(q, kmin, kmax, 7 * 16, T)[0, 0] == 0            # everything selected: nothing to decide
    assert O.near_ties_batch(q, kmin, kmax, 0, T)[0, 0] == 0
    # a second head whose bound is larger on one page takes over there (max over the group's heads)
    q2 = np.zeros((1, 2, 128), np.uint16); q2[0, 0, 0] = bf(1.0); q2[0, 1, 1] = bf(1.0)
    kmin[0, 0, 2, 1] = kmax[0, 0, 2, 1] = bf(5.0)                           # page 2: head 1 sees 5 instead of 1
    assert O.near_ties_batch(q2, kmin, kmax, 3 * 16, T)[0, 0] == 3


def _popcounts(mask):
    return np.vectorize(lambda x: bin(int(x)).count("1"))(mask)


@pytest.mark.parametrize("S,K,mpt,mode", [(8, 4, 1, 0), (8, 7, 1, 0), (16, 4, 1, 0), (4, 1, 1, 1), (8, 2, 0, 0), (8, 8, 1, 0)])
def test_routing_of_pages_completed_during_decoding(S, K, mpt, mode):
    """A decode loop on the checker: a routed prefix, then tokens appended at full width; complete
    pages are routed as they close.  Pinned by (a) the running budget: the routed tokens always hold
    exactly N*K groups (Appendix B.1), the open page S per token; (b) the data: unpacking the store gives
    V with the dropped groups zeroed, for every token, after every step (the in-place compaction moved
    the right bytes); (c) a second construction that never compacts in place: the final masks packed
    from the dense values in one sequential walk; (d) the page rule itself: each completed page's
    masks are those of the (exhaustively pinned) routing rule applied to that page alone; (e) routing the
    closed pages one call at a time or several at once gives the same store."""
    rng = np.random.default_rng(100 + S + K)
    g = 128 // S
    T0, T1 = 16 * 3 + 5, 16 * 9 + 11                      # prefix ends inside a page; 6 pages close during the loop
    v = rng.integers(1, 2 ** 16, size=(T1, 128), dtype=np.uint16)
    sc = np.round(rng.standard_normal((T1, S)).astype(np.float32) * 4) / 4    # ties
    cap = T1 * S
    # prefix: routed up to the last complete page, its open page at full width
    cls = np.ones(T0, np.uint8); cls[16 * 3:] = O.CLS_FULL
    rc, m0 = O.route(sc[:T0], cls, S, K, mpt, mode)
    assert rc == 0
    mask = np.zeros(T1, np.uint16); mask[:T0] = m0
    total, offs0, packed = O.pack(v[:T0], mask[:T0], S, cap)
    offs = np.zeros(T1 + 1, np.uint32); offs[:T0 + 1] = offs0

    def check(length, first_open_page):
        routed = first_open_page * 16
        cnt = _popcounts(mask[:length])
        if mode == 1:
            assert (cnt[:routed] == K).all()
        else:
            assert cnt[:routed].sum() == routed * K                      # M = N*K at every step
            if mpt:
                assert cnt[:routed].min() >= 1
        assert (cnt[routed:length] == S).all()
        assert (np.diff(offs[:length + 1].astype(np.int64)) == cnt).all()
        for t in range(length):                                          # unpack == V with dropped groups removed
            o = int(offs[t])
            for j in range(S):
                if (mask[t] >> j) & 1:
                    np.testing.assert_array_equal(packed[o], v[t, j * g:(j + 1) * g]); o += 1

    length, first_open = T0, 3
    snapshots = {}
    for t in range(T0, T1):                                              # append one token at full width
        mask[t] = (1 << S) - 1
        for j in range(S):
            packed[int(offs[t]) + j] = v[t, j * g:(j + 1) * g]
        offs[t + 1] = offs[t] + S
        length = t + 1
        if length % 16 == 0:
            if length // 16 in (5, 6):                                   # let two pages pile up, route them together
                if length // 16 == 5:
                    continue
            new_total = O.route_new_pages(sc, length, S, first_open, K, mask, offs, packed, mpt, mode)
            assert new_total == int(offs[length])
            first_open = length // 16
            check(length, first_open)
            snapshots[length] = (mask[:length].copy(), packed[:new_total].copy())
    check(length, first_open)
    # (c) + (d): the same final state built without any in-place step
    want = np.zeros(T1, np.uint16); want[:16 * 3] = m0[:16 * 3]
    for p in range(3, T1 // 16):
        rc, mp_ = O.route(sc[16 * p:16 * p + 16], None, S, K, mpt, mode)
        assert rc == 0
        want[16 * p:16 * p + 16] = mp_
    want[(T1 // 16) * 16:] = (1 << S) - 1
    np.testing.assert_array_equal(mask, want)
    total2, offs2, packed2 = O.pack(v, want, S, cap)
    np.testing.assert_array_equal(offs, offs2)
    np.testing.assert_array_equal(packed[:total2], packed2[:total2])
    # refusals leave everything as it was
    before = (mask.copy(), offs.copy(), packed.copy())
    if K < S:
        assert O.route_new_pages(sc, T1, S, 2, K, mask, offs, packed, mpt, mode) == -2  # page 2 is not at full width
    if mode == 0 and mpt == 1:
        m2 = mask.copy(); m2[T1 - 11:] = (1 << S) - 1
        assert O.route_new_pages(sc, T1 - 11 + 16, S, T1 // 16, 0, m2, offs.copy(), packed.copy(), 1, 0) in (-1, -2)
    for a, b in zip(before, (mask, offs, packed)):
        np.testing.assert_array_equal(a, b)
