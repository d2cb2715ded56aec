"""Pins of the fp64 oracle against facts fixed by the paper's definition and by mathematics.

Each test is chosen so that a plausible slip in the oracle (dropped scale, wrong sign in the
exponent, transposed operand, off-by-one in the causal boundary, wrong GQA grouping, wrong
layout offset) fails at least one of them.  None of them re-types the oracle's own formula
with the same routine: they use closed forms, invariances, exhaustive enumeration without the
max subtraction, and a library fp64 softmax attention.
"""
import math

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si

f2b = si.f32_to_bf16_bits
b2f = si.bf16_bits_to_f32


def rnd(rng, *shape, mult=1.0):
    return f2b((mult * rng.standard_normal(shape)).astype(np.float32))


def call(Q, K, V, kv_len, *, Hkv, T=None, scale=0.0):
    B, Hq, T_, d = Q.shape
    kv_len = np.asarray(kv_len, dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(kv_len)]).astype(np.int32)
    return oracle.xattn(Q, K, V, cu, kv_len, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T_, scale=scale)


def test_single_key_returns_its_value():
    rng = np.random.default_rng(0)
    Q = rnd(rng, 2, 4, 1, 8)
    K = rnd(rng, 2 * 2 * 1 * 8)
    V = rnd(rng, 2 * 2 * 1 * 8)
    O, LSE = call(Q, K, V, [1, 1], Hkv=2)
    Vf = b2f(V).reshape(2, 2, 1, 8)
    for b in range(2):
        for h in range(4):
            np.testing.assert_array_equal(O[b, h, 0], Vf[b, h // 2, 0].astype(np.float64))
    # LSE of one key is its score
    Qf, Kf = b2f(Q).astype(np.float64), b2f(K).reshape(2, 2, 1, 8).astype(np.float64)
    want = np.einsum("bhe,bhe->bh", Qf[:, :, 0], np.repeat(Kf[:, :, 0], 2, axis=1)) / math.sqrt(8)
    np.testing.assert_allclose(LSE[:, :, 0], want, rtol=1e-14)


def test_identical_keys_give_prefix_means_under_causal_mask():
    """All scores equal -> uniform weights over the visible keys; with T rows appended at the end
    row t must average exactly keys [0, N-T+t], which pins the mask boundary for every t."""
    rng = np.random.default_rng(1)
    B, Hq, Hkv, d, T, N = 1, 2, 1, 4, 5, 9
    Q = rnd(rng, B, Hq, T, d)
    krow = rnd(rng, d)
    K = np.tile(krow, N)
    V = rnd(rng, N * d)
    O, LSE = call(Q, K, V, [N], Hkv=Hkv)
    Vf = b2f(V).reshape(N, d).astype(np.float64)
    for t in range(T):
        n_vis = N - T + t + 1
        for h in range(Hq):
            np.testing.assert_allclose(O[0, h, t], Vf[:n_vis].mean(axis=0), rtol=1e-14, atol=1e-15)
            s = float(b2f(Q)[0, h, t].astype(np.float64) @ b2f(krow).astype(np.float64)) / math.sqrt(d)
            assert LSE[0, h, t] == pytest.approx(s + math.log(n_vis), rel=1e-13)


def test_selected_rows_of_a_ragged_batch_give_prefix_means_of_their_own_sequence():
    """The row-sampling entry (what the full-size chunk checks and the timed CPU baseline call) on a
    ragged batch of three sequences with a head stride, rows taken from every sequence in scrambled
    order.  Keys are identical inside a (sequence, KV head), so every answer is a closed form: the mean
    of that sequence's, that head's values over keys [0, N_i - T + t], and LSE = score + log(count).
    A slip in the (b, h, t) indexing, in the per-sequence offset or in the GQA head would pick another
    sequence's or head's values, which differ."""
    rng = np.random.default_rng(11)
    B, Hq, Hkv, d, T = 3, 6, 2, 4, 4
    lens = np.array([9, 4, 14], dtype=np.int32)
    cap = 16                                                   # rows per head: spare capacity behind every head
    cu = np.array([0, cap, 2 * cap, 3 * cap], dtype=np.int32)
    Q = rnd(rng, B, Hq, T, d)
    K = rnd(rng, B * Hkv * cap * d)                            # slack rows hold noise
    V = rnd(rng, B * Hkv * cap * d)
    Kv, Vv = K.reshape(B, Hkv, cap, d), V.reshape(B, Hkv, cap, d)
    krows = rnd(rng, B, Hkv, d)
    for b in range(B):
        for c in range(Hkv):
            Kv[b, c, :lens[b]] = krows[b, c]
    rows = [(b, h, t) for b in range(B) for h in range(Hq) for t in range(T)]
    rng.shuffle(rows)
    rows = np.array(rows, dtype=np.int32)
    O, LSE = oracle.xattn_rows(Q, K, V, cu, lens, rows, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, kv_head_stride=cap * d)
    Vf, Qf, Kf = b2f(Vv).astype(np.float64), b2f(Q).astype(np.float64), b2f(krows).astype(np.float64)
    seen = set()
    for k, (b, h, t) in enumerate(rows):
        c = h // (Hq // Hkv)
        n_vis = int(lens[b]) - T + t + 1
        seen.add(b)
        np.testing.assert_allclose(O[k], Vf[b, c, :n_vis].mean(axis=0), rtol=1e-14, atol=1e-15)
        s_ = float(Qf[b, h, t] @ Kf[b, c]) / math.sqrt(d)
        assert LSE[k] == pytest.approx(s_ + math.log(n_vis), rel=1e-13)
    assert seen == {0, 1, 2}
    # and it is the same routine as the full evaluation, row for row
    Of, Lf = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T, kv_head_stride=cap * d)
    for k, (b, h, t) in enumerate(rows):
        np.testing.assert_array_equal(O[k], Of[b, h, t])
        assert LSE[k] == Lf[b, h, t]


def test_zero_query_gives_plain_mean_and_log_n():
    rng = np.random.default_rng(2)
    N, d = 37, 16
    Q = np.zeros((1, 3, 1, d), dtype=np.uint16)
    K, V = rnd(rng, 3 * N * d), rnd(rng, 3 * N * d)
    O, LSE = call(Q, K, V, [N], Hkv=3)
    Vf = b2f(V).reshape(3, N, d).astype(np.float64)
    np.testing.assert_allclose(O[0, :, 0], Vf.mean(axis=1), rtol=1e-14)
    np.testing.assert_allclose(LSE, math.log(N), rtol=1e-14)


def test_permuting_key_value_pairs_changes_nothing():
    rng = np.random.default_rng(3)
    N, d, Hkv = 50, 8, 2
    Q = rnd(rng, 1, 4, 1, d)
    K, V = rnd(rng, Hkv, N, d), rnd(rng, Hkv, N, d)
    O1, L1 = call(Q, K, V, [N], Hkv=Hkv)
    perm = rng.permutation(N)
    O2, L2 = call(Q, K[:, perm], V[:, perm], [N], Hkv=Hkv)
    np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(L1, L2, rtol=1e-13)


def test_split_and_lse_merge_equals_unsplit():
    rng = np.random.default_rng(4)
    B, Hq, Hkv, d, T = 2, 6, 2, 16, 3
    lens = np.array([70, 41], dtype=np.int32)
    cu = np.array([0, 70, 111], dtype=np.int32)
    Q = rnd(rng, B, Hq, T, d, mult=2.0)
    K, V = rnd(rng, 111 * Hkv * d), rnd(rng, 111 * Hkv * d)
    kw = dict(B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
    O, L = oracle.xattn(Q, K, V, cu, lens, **kw)
    for cuts in ([], [1], [10, 10, 33], [5, 40, 41, 69, 200], list(range(0, 80, 7))):
        O2, L2 = oracle.xattn_split_merge(Q, K, V, cu, lens, cuts, **kw)
        np.testing.assert_allclose(O2, O, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(L2, L, rtol=1e-13)


def test_brute_force_enumeration_without_max_subtraction():
    """Tiny shapes, every term of sum_j e^{s_j} v_j / sum_j e^{s_j} written out with Python floats
    via math.fsum, no stabilisation, independent indexing of the packed layout."""
    rng = np.random.default_rng(5)
    B, Hq, Hkv, d, T = 2, 4, 2, 2, 2
    lens = [4, 3]
    cu = [0, 4, 7]
    Q = rnd(rng, B, Hq, T, d)
    K, V = rnd(rng, 7 * Hkv * d), rnd(rng, 7 * Hkv * d)
    O, LSE = call(Q, K, V, lens, Hkv=Hkv, scale=0.37)
    Qf, Kf, Vf = b2f(Q).astype(np.float64), b2f(K).astype(np.float64), b2f(V).astype(np.float64)
    G = Hq // Hkv
    for b in range(B):
        N = lens[b]
        for h in range(Hq):
            c = h // G
            base = cu[b] * Hkv * d + c * N * d
            for t in range(T):
                vis = N - T + t + 1
                ws = []
                for j in range(vis):
                    s = 0.37 * math.fsum(Qf[b, h, t, e] * Kf[base + j * d + e] for e in range(d))
                    ws.append(math.exp(s))
                den = math.fsum(ws)
                for e in range(d):
                    num = math.fsum(ws[j] * Vf[base + j * d + e] for j in range(vis))
                    assert O[b, h, t, e] == pytest.approx(num / den, rel=1e-13, abs=1e-15)
                assert LSE[b, h, t] == pytest.approx(math.log(den), rel=1e-13, abs=1e-14)


def test_two_keys_logistic_closed_form():
    rng = np.random.default_rng(6)
    d = 8
    Q, K, V = rnd(rng, 1, 1, 1, d), rnd(rng, 2, d), rnd(rng, 2, d)
    O, _ = call(Q, K, V, [2], Hkv=1)
    q, k, v = (b2f(x).astype(np.float64) for x in (Q, K, V))
    s = (k @ q[0, 0, 0]) / math.sqrt(d)
    sig = 1.0 / (1.0 + math.exp(-(s[0] - s[1])))
    np.testing.assert_allclose(O[0, 0, 0], sig * v[0] + (1 - sig) * v[1], rtol=1e-13)


def test_default_scale_is_inverse_sqrt_d_and_scale_argument_is_used():
    rng = np.random.default_rng(7)
    d, N = 16, 12
    Q, K, V = rnd(rng, 1, 1, 1, d), rnd(rng, N, d), rnd(rng, N, d)
    O_def, L_def = call(Q, K, V, [N], Hkv=1)
    O_exp, L_exp = call(Q, K, V, [N], Hkv=1, scale=0.25)
    np.testing.assert_array_equal(O_def, O_exp)
    O_other, _ = call(Q, K, V, [N], Hkv=1, scale=1.0)
    assert np.abs(O_other - O_def).max() > 1e-3


def test_affine_map_of_values_and_range_bound():
    """V -> 2V + 1 (exact in bf16 for these small-integer values) gives 2O + 1; every output
    channel lies inside the range of the visible values."""
    rng = np.random.default_rng(8)
    N, d = 33, 8
    Q, K = rnd(rng, 1, 2, 1, d), rnd(rng, N, d)
    Vi = rng.integers(-20, 20, size=(N, d)).astype(np.float32)
    O1, _ = call(Q, K, f2b(Vi), [N], Hkv=1)
    O2, _ = call(Q, K, f2b(2 * Vi + 1), [N], Hkv=1)
    np.testing.assert_allclose(O2, 2 * O1 + 1, rtol=1e-13, atol=1e-13)
    assert (O1 <= Vi.max(axis=0) + 1e-12).all() and (O1 >= Vi.min(axis=0) - 1e-12).all()


def test_shifting_all_keys_by_a_constant_vector_changes_nothing():
    rng = np.random.default_rng(9)
    N, d = 21, 4
    Q = rnd(rng, 1, 1, 1, d)
    Ki = rng.integers(-8, 8, size=(N, d)).astype(np.float32)
    V = rnd(rng, N, d)
    shift = np.array([3, -2, 5, 1], dtype=np.float32)
    O1, L1 = call(Q, f2b(Ki), V, [N], Hkv=1)
    O2, L2 = call(Q, f2b(Ki + shift), V, [N], Hkv=1)
    np.testing.assert_allclose(O1, O2, rtol=1e-12, atol=1e-14)
    delta = float(b2f(Q)[0, 0, 0].astype(np.float64) @ shift.astype(np.float64)) / math.sqrt(d)
    np.testing.assert_allclose(L2 - L1, delta, rtol=1e-12)


def test_gqa_equals_mha_with_repeated_kv_heads():
    """Query head h reads KV head h // G (contiguous groups)."""
    rng = np.random.default_rng(10)
    N, d, Hq, Hkv = 19, 8, 6, 2
    Q = rnd(rng, 1, Hq, 1, d)
    K, V = rnd(rng, Hkv, N, d), rnd(rng, Hkv, N, d)
    O_g, L_g = call(Q, K, V, [N], Hkv=Hkv)
    O_m, L_m = call(Q, np.repeat(K, 3, axis=0), np.repeat(V, 3, axis=0), [N], Hkv=Hq)
    np.testing.assert_array_equal(O_g, O_m)
    np.testing.assert_array_equal(L_g, L_m)


def test_chunk_row_equals_single_query_call_on_truncated_cache():
    rng = np.random.default_rng(11)
    N, d, T, Hq, Hkv = 30, 8, 4, 4, 2
    Q = rnd(rng, 1, Hq, T, d)
    K, V = rnd(rng, Hkv, N, d), rnd(rng, Hkv, N, d)
    O, L = call(Q, K, V, [N], Hkv=Hkv)
    for t in range(T):
        n = N - T + t + 1
        O1, L1 = call(Q[:, :, t:t + 1], K[:, :n], V[:, :n], [n], Hkv=Hkv)
        np.testing.assert_array_equal(O[:, :, t], O1[:, :, 0])
        np.testing.assert_array_equal(L[:, :, t], L1[:, :, 0])


def test_rows_beyond_the_cache_see_nothing():
    rng = np.random.default_rng(12)
    d, T, N = 4, 5, 3     # rows t = 0, 1 have no visible key
    Q, K, V = rnd(rng, 1, 1, T, d), rnd(rng, N, d), rnd(rng, N, d)
    O, L = call(Q, K, V, [N], Hkv=1)
    assert (O[0, 0, :2] == 0).all() and np.isneginf(L[0, 0, :2]).all()
    np.testing.assert_array_equal(O[0, 0, 2], b2f(V)[0].astype(np.float64))
    assert np.isfinite(O).all()


def test_empty_sequence_in_a_batch():
    rng = np.random.default_rng(13)
    d = 4
    Q, K, V = rnd(rng, 2, 2, 1, d), rnd(rng, 2 * 5 * d), rnd(rng, 2 * 5 * d)
    O, L = call(Q, K, V, [0, 5], Hkv=2)
    assert (O[0] == 0).all() and np.isneginf(L[0]).all() and np.isfinite(L[1]).all()


@pytest.mark.parametrize("T", [1, 7])
def test_library_fp64_attention_on_small_ragged_batch(T):
    """torch's scaled_dot_product_attention in fp64 with an explicit boolean mask is the same
    textbook routine; the packed head-major layout is unpacked here by independent indexing."""
    rng = np.random.default_rng(14)
    B, Hq, Hkv, d = 3, 6, 2, 16
    lens = np.array([23, 9, 40], dtype=np.int32)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    Q = rnd(rng, B, Hq, T, d)
    K, V = rnd(rng, int(cu[-1]) * Hkv * d), rnd(rng, int(cu[-1]) * Hkv * d)
    O, L = oracle.xattn(Q, K, V, cu, lens, B=B, Hq=Hq, Hkv=Hkv, d=d, T=T)
    for b in range(B):
        N = int(lens[b])
        sl = slice(int(cu[b]) * Hkv * d, int(cu[b + 1]) * Hkv * d)
        k = torch.from_numpy(b2f(K[sl]).reshape(Hkv, N, d)).double().repeat_interleave(Hq // Hkv, 0)
        v = torch.from_numpy(b2f(V[sl]).reshape(Hkv, N, d)).double().repeat_interleave(Hq // Hkv, 0)
        q = torch.from_numpy(b2f(Q[b])).double()
        mask = torch.arange(N)[None, :] <= (N - T + torch.arange(T))[:, None]
        ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, attn_mask=mask)
        np.testing.assert_allclose(O[b], ref.numpy(), rtol=1e-11, atol=1e-13)
        s = (q @ k.transpose(1, 2)) / math.sqrt(d)
        lse = torch.logsumexp(s.masked_fill(~mask, -math.inf), dim=-1)
        np.testing.assert_allclose(L[b], lse.numpy(), rtol=1e-12)


def test_head_stride_layout_matches_tight_layout():
    """A cache with spare capacity per head (stride > N*d) gives the same result."""
    rng = np.random.default_rng(15)
    N, cap, d, Hkv = 11, 16, 8, 2
    Q = rnd(rng, 1, 4, 1, d)
    K, V = rnd(rng, Hkv, N, d), rnd(rng, Hkv, N, d)
    Kc = rnd(rng, Hkv, cap, d)
    Vc = rnd(rng, Hkv, cap, d)
    Kc[:, :N], Vc[:, :N] = K, V
    O1, L1 = call(Q, K, V, [N], Hkv=Hkv)
    lens = np.array([N], dtype=np.int32)
    cu = np.array([0, cap], dtype=np.int32)
    O2, L2 = oracle.xattn(Q, Kc, Vc, cu, lens, B=1, Hq=4, Hkv=Hkv, d=d, T=1, kv_head_stride=cap * d)
    np.testing.assert_array_equal(O1, O2)
    np.testing.assert_array_equal(L1, L2)


def test_one_hot_selection_is_exact():
    """A key whose score leads by > 700 nats takes all the weight even in fp64."""
    d, N = 16, 40
    q = np.full((1, 1, 1, d), 16.0, dtype=np.float32)
    K = np.zeros((N, d), dtype=np.float32)
    K[29] = 16.0
    rng = np.random.default_rng(16)
    V = rnd(rng, N, d)
    O, L = call(f2b(q), f2b(K), V, [N], Hkv=1)
    np.testing.assert_array_equal(O[0, 0, 0], b2f(V)[29].astype(np.float64))
    assert L[0, 0, 0] == pytest.approx(16 * 16 * d / math.sqrt(d))


def test_combine_oracle_against_direct_merge():
    """Merging normalised partials by LSE: checked against pooling the un-normalised sums."""
    rng = np.random.default_rng(17)
    rows, S, d = 5, 4, 8
    lse = rng.standard_normal((rows, S)).astype(np.float32) * 3
    lse[1, 2] = -np.inf
    lse[3, :] = -np.inf
    po = rng.standard_normal((rows, S, d)).astype(np.float32)
    O, L = oracle.combine(po, lse)
    for r in range(rows):
        w = [math.exp(float(x)) if np.isfinite(x) else 0.0 for x in lse[r]]
        tot = math.fsum(w)
        if tot == 0:
            assert (O[r] == 0).all() and np.isneginf(L[r])
            continue
        want = sum(w[s] * po[r, s].astype(np.float64) for s in range(S)) / tot
        np.testing.assert_allclose(O[r], want, rtol=1e-12, atol=1e-14)
        assert L[r] == pytest.approx(math.log(tot), rel=1e-12, abs=1e-13)


def test_combine_single_nonempty_piece_is_pass_through():
    rng = np.random.default_rng(18)
    po = rng.standard_normal((3, 4, 8)).astype(np.float32)
    lse = np.full((3, 4), -np.inf, dtype=np.float32)
    lse[0, 0], lse[1, 3], lse[2, 1] = 0.5, -7.0, 88.0
    O, L = oracle.combine(po, lse)
    np.testing.assert_array_equal(O[0], po[0, 0].astype(np.float64))
    np.testing.assert_array_equal(O[1], po[1, 3].astype(np.float64))
    np.testing.assert_array_equal(O[2], po[2, 1].astype(np.float64))
    np.testing.assert_array_equal(L, np.array([0.5, -7.0, 88.0]))


def test_planted_mistakes_are_caught():
    """The pins bite: an off-by-one causal boundary and a wrong head grouping, planted in a copy
    of the expected values, do not match the oracle."""
    rng = np.random.default_rng(19)
    N, d, T = 9, 4, 3
    Q = rnd(rng, 1, 2, T, d)
    K = np.tile(rnd(rng, d), N)
    V = rnd(rng, N * d)
    O, _ = call(Q, K, V, [N], Hkv=1)
    Vf = b2f(V).reshape(N, d).astype(np.float64)
    wrong = Vf[: N - T + 0].mean(axis=0)          # excludes the row's own position
    assert np.abs(O[0, 0, 0] - wrong).max() > 1e-6
    Q6 = rnd(rng, 1, 6, 1, d)
    K2, V2 = rnd(rng, 2, N, d), rnd(rng, 2, N, d)
    Og, _ = call(Q6, K2, V2, [N], Hkv=2)
    Oi, _ = call(Q6, np.tile(K2, (3, 1, 1)), np.tile(V2, (3, 1, 1)), [N], Hkv=6)  # h % Hkv grouping
    assert np.abs(Og - Oi).max() > 1e-6
