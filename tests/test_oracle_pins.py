"""Pins for the CPU oracle: each part is tied to something other than itself -- a closed form, an
invariant, a library routine on a special case, a hand-worked value, the paper's own constants,
or a brute-force restatement on tiny inputs -- so that a dropped term, a wrong sign or index, or a
transposed operand in the oracle fails at least one test here.  No GPU is used."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import kvr_oracle as orc
from paper_2512_17917_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
P = 2 ** 31 - 1


def _rand(shape, seed, scale=1.0):
    return (np.random.default_rng(seed).standard_normal(shape) * scale).astype(np.float32)


# ------------------------------------------------------------------------------------ hashing
def test_hash_hand_worked_examples():
    """Values derived by hand from the hash family's definition (tests/golden)."""
    n = 0
    for line in open(os.path.join(GOLDEN, "hash_worked_examples.txt")):
        line = line.split("#")[0].split()
        if not line:
            continue
        kind, mix = line[0], bool(int(line[1]))
        A, C, J, b, want = (int(x) for x in line[2:7])
        if kind == "bucket":
            seeds = np.array([[A, C, 1, 0]], np.uint32)
            got = orc.bucket_sign([J], seeds, b, mix)[0][0, 0]
        else:
            seeds = np.array([[1, 0, A, C]], np.uint32)
            got = orc.bucket_sign([J], seeds, 5, mix)[1][0, 0]
        assert got == want, (kind, mix, A, C, J, b)
        n += 1
    assert n >= 20


def test_hash_identity_seed_is_mod_b():
    """Without index scrambling A=1, C=0 gives h(J) = J mod b; A'=0, C'=0 gives g = +1."""
    J = np.arange(0, 5000, dtype=np.int32)
    seeds = np.array([[1, 0, 0, 0]] * 3, np.uint32)
    for b in (1, 6, 273, 8000):
        bucket, sign = orc.bucket_sign(J, seeds, b, mix=False)
        assert (bucket == (J % b)[None, :]).all()
        assert (sign == 1).all()


def test_hash_rows_differ_and_are_roughly_uniform():
    """Random seeds over consecutive token indices behave like random hashing: even occupancy
    (chi-square), per-cell sign sums of variance ~ cell size, two-row pair collisions at the
    a^2/(2 b^2) rate, and rows that are distinct functions."""
    b, n = 64, 64 * 400
    for seed in (99, 100, 101):
        seeds = synth.hash_seeds(seed, 3)
        bucket, sign = orc.bucket_sign(np.arange(n), seeds, b)
        for i in range(3):
            cnt = np.bincount(bucket[i], minlength=b)
            chi2 = ((cnt - n / b) ** 2 / (n / b)).sum()
            assert 0.5 * b < chi2 < 1.6 * b, chi2          # mean b-1, sd sqrt(2b)
            cell_sum = np.bincount(bucket[i], weights=sign[i].astype(np.float64), minlength=b)
            assert 0.6 < (cell_sum ** 2).mean() / (n / b) < 1.5
        for i, k in ((0, 1), (0, 2), (1, 2)):
            c = np.bincount(bucket[i].astype(np.int64) * b + bucket[k])
            pairs = (c * (c - 1) // 2).sum()
            assert 0.85 < pairs / (n * (n - 1) / 2 / b / b) < 1.15
            assert (bucket[i] != bucket[k]).mean() > 0.9
        assert 0.4 < (sign[0] != sign[1]).mean() < 0.6


# ------------------------------------------------------------------------------------ scoring
def test_scores_match_library_softmax_column_sum():
    n_inst, GW, N, D = 3, 12, 57, 16
    Q, K = _rand((n_inst, GW, D), 1), _rand((n_inst, N, D), 2)
    s = orc.scores(Q, K)
    tq, tk = torch.from_numpy(Q).double(), torch.from_numpy(K).double()
    want = torch.softmax(tq @ tk.transpose(1, 2) / math.sqrt(D), dim=-1).sum(dim=1).numpy()
    np.testing.assert_allclose(s, want, rtol=1e-12, atol=1e-14)


def test_scores_rows_sum_to_one_and_scale_matters():
    """Every softmax row sums to 1, so the scores sum to G*W; the 1/sqrt(d) scale is not 1."""
    Q, K = _rand((2, 8, 32), 3), _rand((2, 100, 32), 4)
    s = orc.scores(Q, K)
    np.testing.assert_allclose(s.sum(axis=1), 8.0, rtol=1e-12)
    s1 = orc.scores(Q, K, scale=1.0)
    assert np.abs(s - s1).max() > 1e-2


def test_scores_transposition_would_be_caught():
    """Non-square case: token j's score moves with K row j (a one-hot-ish key row that matches
    every query gets nearly all the mass)."""
    D, N = 8, 20
    Q = np.ones((1, 4, D), np.float32)
    K = np.zeros((1, N, D), np.float32)
    K[0, 13, :] = 6.0
    s = orc.scores(Q, K)
    assert s[0].argmax() == 13 and s[0, 13] > 3.99


# ---------------------------------------------------------------------------------- selection
def _select_by_full_sort(s, R, n_recent):
    N = len(s)
    n_cand = N - n_recent
    order = np.lexsort((np.arange(n_cand), -s[:n_cand].astype(np.float64)))   # score desc, index asc
    keep = np.zeros(N, bool)
    keep[order[: R - n_recent]] = True
    keep[n_cand:] = True
    return np.nonzero(keep)[0], np.nonzero(~keep)[0]


@pytest.mark.parametrize("N,R,n_recent", [(50, 10, 0), (64, 17, 8), (33, 33, 0), (33, 0, 0), (40, 12, 12)])
def test_select_equals_full_sort_with_ties(N, R, n_recent):
    rng = np.random.default_rng(N + R)
    s = rng.integers(0, 6, size=(4, N)).astype(np.float32) / 8      # many exact ties
    ret, cmp_ = orc.select(s, R, n_recent)
    for u in range(4):
        wr, wc = _select_by_full_sort(s[u], R, n_recent)
        assert (ret[u] == wr).all() and (cmp_[u] == wc).all()


def test_select_degenerate_budgets():
    s = _rand((2, 30), 5) ** 2
    ret, cmp_ = orc.select(s, 30, 0)
    assert (ret == np.arange(30)).all() and cmp_.shape == (2, 0)
    ret, cmp_ = orc.select(s, 7, 7)                                   # all budget to Recent
    assert (ret == np.arange(23, 30)).all()
    ret, _ = orc.select(s, 1, 0)
    assert (ret[:, 0] == s.argmax(axis=1)).all()


# ------------------------------------------------------------------------------------- insert
def _setup(n_inst=2, N=300, D=8, seed=11):
    return _rand((n_inst, N, D), seed), _rand((n_inst, N, D), seed + 1)


def test_insert_is_linear():
    """sketch(S1 u S2) = sketch(S1) + sketch(S2) for disjoint token sets."""
    K, V = _setup()
    seeds, b = synth.hash_seeds(5), 13
    idx = np.arange(300, dtype=np.int32)[None].repeat(2, 0)
    full = orc.insert(K, V, idx, seeds, b)
    a = orc.insert(K, V, idx[:, :111], seeds, b)
    c = orc.insert(K, V, idx[:, 111:], seeds, b)
    np.testing.assert_allclose(full, a + c, rtol=0, atol=1e-12)


def test_insert_conservation_per_row_keys_unsigned_values_signed():
    """Each row receives every token once: sum of key cells = sum of keys (no sign on keys);
    sum of value cells = sum of g_i(J) * values."""
    K, V = _setup()
    seeds, b = synth.hash_seeds(6), 9
    idx = np.arange(0, 300, 2, dtype=np.int32)[None].repeat(2, 0)
    cells = orc.insert(K, V, idx, seeds, b)
    _, sign = orc.bucket_sign(idx[0], seeds, b)
    for i in range(3):
        np.testing.assert_allclose(cells[:, i, :, 0, :].sum(axis=1), K[:, idx[0]].astype(np.float64).sum(axis=1), atol=1e-10)
        want_v = (V[:, idx[0]].astype(np.float64) * sign[i][None, :, None]).sum(axis=1)
        np.testing.assert_allclose(cells[:, i, :, 1, :].sum(axis=1), want_v, atol=1e-10)
    assert (sign == -1).any() and (sign == 1).any()


def test_insert_single_token_lands_in_its_cells_only():
    K, V = _setup(1, 50, 4)
    seeds, b = synth.hash_seeds(7), 11
    J = 37
    cells = orc.insert(K, V, np.array([[J]], np.int32), seeds, b)
    bucket, sign = orc.bucket_sign([J], seeds, b)
    for i in range(3):
        for c in range(b):
            if c == bucket[i, 0]:
                np.testing.assert_array_equal(cells[0, i, c, 0], K[0, J].astype(np.float64))
                np.testing.assert_array_equal(cells[0, i, c, 1], V[0, J].astype(np.float64) * sign[i, 0])
            else:
                assert not cells[0, i, c].any()


# -------------------------------------------------------------------------------------- query
def test_query_injective_hashing_is_exact():
    """b >= N with h(J) = J: no collisions, so every token comes back exactly (g*g = 1)."""
    K, V = _setup(2, 120, 16)
    seeds = synth.injective_seeds()
    idx = np.arange(120, dtype=np.int32)[None].repeat(2, 0)
    cells = orc.insert(K, V, idx, seeds, 128, mix=False)
    Kt, Vt = orc.query(cells, idx, seeds, mix=False)
    np.testing.assert_array_equal(Kt, K.astype(np.float64))
    np.testing.assert_array_equal(Vt, V.astype(np.float64))
    assert (orc.bucket_sign(idx[0], seeds, 128, mix=False)[1] == -1).any()


def test_query_single_row_is_direct_lookup():
    K, V = _setup(1, 60, 4)
    seeds, b = synth.hash_seeds(8, r=1), 7
    idx = np.arange(60, dtype=np.int32)[None]
    cells = orc.insert(K, V, idx, seeds, b)
    bucket, sign = orc.bucket_sign(idx[0], seeds, b)
    Kt, Vt = orc.query(cells, idx, seeds)
    np.testing.assert_array_equal(Kt[0], cells[0, 0, bucket[0], 0])
    np.testing.assert_array_equal(Vt[0], cells[0, 0, bucket[0], 1] * sign[0][:, None])


def test_query_is_elementwise_middle_of_three():
    K, V = _setup(1, 200, 6)
    seeds, b = synth.hash_seeds(9), 5
    idx = np.arange(200, dtype=np.int32)[None]
    cells = orc.insert(K, V, idx, seeds, b)
    bucket, sign = orc.bucket_sign(idx[0], seeds, b)
    Kt, Vt = orc.query(cells, idx, seeds)
    rows = np.arange(3)[:, None]
    np.testing.assert_array_equal(Kt[0], np.median(cells[0, rows, bucket, 0], axis=0))
    np.testing.assert_array_equal(Vt[0], np.median(cells[0, rows, bucket, 1] * sign[:, :, None], axis=0))


def test_query_error_matches_median_of_three_normals_constant():
    """i.i.d. N(0,1) tokens: each of a token's three cells holds the token plus ~(a-1)/b others, so
    the reconstruction error is the median of three ~N(0, lam) noises: variance (1 - sqrt(3)/pi) lam
    = 0.4487 lam (Lemma 2 prints 0.448), not lam (one row) nor lam/3 (a mean), and below the
    paper's bound a*pi/(r*b) (Mathematical Analysis section)."""
    a, b, D = 6000, 120, 64
    K, V = _rand((1, a, D), 21), _rand((1, a, D), 22)
    seeds = synth.hash_seeds(23)
    idx = np.arange(a, dtype=np.int32)[None]
    cells = orc.insert(K, V, idx, seeds, b)
    Kt, Vt = orc.query(cells, idx, seeds)
    lam = (a - 1) / b
    c = 1 - math.sqrt(3) / math.pi
    assert abs(c - 0.448) < 1e-3
    for X, Xt in ((K, Kt), (V, Vt)):
        mse = ((Xt - X) ** 2).mean()
        assert abs(mse / (c * lam) - 1) < 0.05, mse / lam
        assert mse < a * math.pi / (3 * b)


def test_values_unbiased_keys_not():
    """Inputs with mean 1: the +-1 coefficients make the value estimate unbiased (Lemma 3), while
    the unsigned key cells carry the collision mass (bias ~ (a-1)/b)."""
    a, b, D = 3000, 100, 32
    K, V = _rand((1, a, D), 31) + 1, _rand((1, a, D), 32) + 1
    seeds = synth.hash_seeds(33)
    idx = np.arange(a, dtype=np.int32)[None]
    cells = orc.insert(K, V, idx, seeds, b)
    Kt, Vt = orc.query(cells, idx, seeds)
    lam = (a - 1) / b
    assert abs((Vt - V).mean()) < 0.15                 # sd of the mean ~ sqrt(0.45*2*lam/(a*D)) ~ 0.02
    assert abs((Kt - K).mean() / lam - 1) < 0.1


# ------------------------------------------------------------------------------------- decode
def _sdpa(q, K, V):
    tq, tk, tv = (torch.from_numpy(x).double() for x in (q, K, V))
    return torch.nn.functional.scaled_dot_product_attention(tq, tk, tv).numpy()


def test_decode_full_budget_is_textbook_attention():
    """100 % budget: nothing is compressed and the output is ordinary softmax attention."""
    n_inst, G, N, D = 2, 4, 90, 16
    q, K, V = _rand((n_inst, G, D), 41), _rand((n_inst, N, D), 42, 1.5), _rand((n_inst, N, D), 43)
    seeds, b = synth.hash_seeds(44), 5
    ret = np.arange(N, dtype=np.int32)[None].repeat(n_inst, 0)
    cells = np.zeros((n_inst, 3, b, 2, D))
    out = orc.decode(q, K, V, ret, cells, N, seeds)
    np.testing.assert_allclose(out, _sdpa(q, K, V), rtol=1e-12, atol=1e-13)


def test_decode_injective_sketch_is_textbook_attention_at_any_budget():
    """With collision-free hashing the rebuilt cache equals the original, so attention over
    retained + reconstructed tokens equals full attention whatever the budget."""
    n_inst, G, N, D = 2, 4, 70, 8
    Q = _rand((n_inst, 8, D), 50)
    q, K, V = _rand((n_inst, G, D), 51), _rand((n_inst, N, D), 52), _rand((n_inst, N, D), 53)
    seeds = synth.injective_seeds()
    c = orc.compress(Q, K, V, R=20, n_recent=5, seeds=seeds, b=80, mix=False)
    out = orc.decode(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds, mix=False)
    np.testing.assert_allclose(out, _sdpa(q, K, V), rtol=1e-12, atol=1e-13)


def test_decode_is_invariant_to_order_of_retained_rows():
    n_inst, G, N, D = 1, 4, 60, 8
    Q = _rand((n_inst, 8, D), 60)
    q, K, V = _rand((n_inst, G, D), 61), _rand((n_inst, N, D), 62), _rand((n_inst, N, D), 63)
    seeds, b = synth.hash_seeds(64), 4
    c = orc.compress(Q, K, V, R=15, n_recent=0, seeds=seeds, b=b)
    out = orc.decode(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds)
    perm = np.random.default_rng(0).permutation(15)
    out2 = orc.decode(q, c["Kr"][:, perm], c["Vr"][:, perm], c["ret_idx"][:, perm], c["cells"], N, seeds)
    np.testing.assert_allclose(out, out2, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------- brute force of the whole path
def _brute_force(Q, K, V, q, R, n_recent, seeds, b):
    """Algorithms 1-4 and the attention formula restated with Python loops and dictionaries for
    one head-instance (tiny sizes only)."""
    N, D = K.shape
    sc = 1.0 / math.sqrt(D)
    s = np.zeros(N)
    for row in Q.astype(np.float64):
        e = np.array([math.exp(sc * sum(row[d] * float(K[j, d]) for d in range(D))) for j in range(N)])
        s += e / e.sum()
    s32 = s.astype(np.float32)
    cand = sorted(range(N - n_recent), key=lambda j: (-float(s32[j]), j))
    keep = set(cand[: R - n_recent]) | set(range(N - n_recent, N))
    def m(J):                                  # 32-bit scrambling bijection of the index
        x = J & 0xFFFFFFFF
        x ^= x >> 16
        x = (x * 0x85EBCA6B) & 0xFFFFFFFF
        x ^= x >> 13
        x = (x * 0xC2B2AE35) & 0xFFFFFFFF
        return x ^ (x >> 16)

    h = lambda i, J: ((int(seeds[i, 0]) * m(J) + int(seeds[i, 1])) % P) % b
    g = lambda i, J: 1 - 2 * (((int(seeds[i, 2]) * m(J) + int(seeds[i, 3])) % P) & 1)
    cell = {}
    for J in range(N):
        if J in keep:
            continue
        for i in range(3):
            ck, cv = cell.setdefault((i, h(i, J)), (np.zeros(D), np.zeros(D)))
            ck += K[J]
            cv += g(i, J) * V[J].astype(np.float64)
    Kf, Vf = np.zeros((N, D)), np.zeros((N, D))
    for J in range(N):
        if J in keep:
            Kf[J], Vf[J] = K[J], V[J]
        else:
            ks = [cell[(i, h(i, J))][0] for i in range(3)]
            vs = [g(i, J) * cell[(i, h(i, J))][1] for i in range(3)]
            for d in range(D):
                Kf[J, d] = sorted(x[d] for x in ks)[1]
                Vf[J, d] = sorted(x[d] for x in vs)[1]
    out = np.zeros((q.shape[0], D))
    for gi, qq in enumerate(q.astype(np.float64)):
        e = np.exp(sc * (Kf @ qq))
        out[gi] = (e / e.sum()) @ Vf
    return s, sorted(keep), out


@pytest.mark.parametrize("N,R,n_recent,b", [(24, 6, 0, 3), (31, 9, 4, 2), (17, 1, 1, 1)])
def test_whole_path_against_brute_force(N, R, n_recent, b):
    D, G, W = 4, 2, 3
    Q = _rand((1, G * W, D), 70 + N)
    q, K, V = _rand((1, G, D), 71 + N), _rand((1, N, D), 72 + N, 2.0), _rand((1, N, D), 73 + N)
    seeds = synth.hash_seeds(74 + N)
    c = orc.compress(Q, K, V, R=R, n_recent=n_recent, seeds=seeds, b=b)
    out = orc.decode(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds)
    s, keep, want = _brute_force(Q[0], K[0], V[0], q[0], R, n_recent, seeds, b)
    np.testing.assert_allclose(c["scores64"][0], s, rtol=1e-12)
    assert list(c["ret_idx"][0]) == keep
    np.testing.assert_allclose(out[0], want, rtol=1e-11, atol=1e-13)


def test_forced_selection_is_honoured():
    N, D = 40, 8
    Q, K, V = _rand((1, 4, D), 80), _rand((1, N, D), 81), _rand((1, N, D), 82)
    seeds = synth.hash_seeds(83)
    forced = np.arange(0, 40, 4, dtype=np.int32)[None]
    c = orc.compress(Q, K, V, R=10, n_recent=0, seeds=seeds, b=3, forced_ret_idx=forced)
    assert (c["ret_idx"] == forced).all()
    assert sorted(set(c["cmp_idx"][0]) | set(forced[0])) == list(range(N))
    np.testing.assert_array_equal(c["cells"], orc.insert(K, V, c["cmp_idx"], seeds, 3))


# ------------------------------------------------- attention mass and the overflow step (streaming)
def test_decode_mass_is_library_softmax_column_sum_and_sums_to_G():
    """100 % budget: the mass of a token is the sum over the G heads of the softmax probability a
    library softmax gives it; in general the masses of all tokens add up to G."""
    n_inst, G, N, D = 2, 4, 80, 16
    q, K, V = _rand((n_inst, G, D), 71), _rand((n_inst, N, D), 72, 1.5), _rand((n_inst, N, D), 73)
    seeds, b = synth.hash_seeds(74), 5
    ret = np.arange(N, dtype=np.int32)[None].repeat(n_inst, 0)
    mass = orc.decode_mass(q, K, V, ret, np.zeros((n_inst, 3, b, 2, D)), N, seeds)
    logits = torch.einsum("ugd,ujd->ugj", torch.from_numpy(q).double(), torch.from_numpy(K).double()) / math.sqrt(D)
    want = torch.softmax(logits, dim=-1).sum(dim=1).numpy()
    np.testing.assert_allclose(mass, want, rtol=1e-12, atol=1e-14)
    Q = _rand((n_inst, 8, D), 75)
    c = orc.compress(Q, K, V, R=20, n_recent=3, seeds=seeds, b=b)
    mass2 = orc.decode_mass(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds)
    np.testing.assert_allclose(mass2.sum(axis=1), G, rtol=1e-12)
    assert (mass2 >= 0).all()


def test_decode_mass_weights_reproduce_the_decode_output_for_one_head():
    """G = 1: out = sum_j mass[j] * v_j over the rebuilt cache (exact rows and Algorithm 2 rows)."""
    n_inst, N, D = 1, 50, 8
    Q = _rand((n_inst, 4, D), 80)
    q, K, V = _rand((n_inst, 1, D), 81), _rand((n_inst, N, D), 82), _rand((n_inst, N, D), 83)
    seeds, b = synth.hash_seeds(84), 3
    c = orc.compress(Q, K, V, R=10, n_recent=2, seeds=seeds, b=b)
    mass = orc.decode_mass(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds)
    out = orc.decode(q, c["Kr"], c["Vr"], c["ret_idx"], c["cells"], N, seeds)
    Vfull = np.empty((N, D))
    Vfull[c["ret_idx"][0]] = c["Vr"][0]
    _, Vt = orc.query(c["cells"], c["cmp_idx"], seeds)
    Vfull[c["cmp_idx"][0]] = Vt[0]
    np.testing.assert_allclose(out[0, 0], mass[0] @ Vfull, rtol=1e-11, atol=1e-13)


def test_insert_rows_equals_insert_by_index():
    n_inst, N, D, b = 2, 40, 8, 4
    K, V = _rand((n_inst, N, D), 90), _rand((n_inst, N, D), 91)
    seeds = synth.hash_seeds(92)
    idx = np.array([[3, 7, 20, 39], [0, 1, 2, 33]], np.int32)
    want = orc.insert(K, V, idx, seeds, b)
    rows_k = np.take_along_axis(K, idx[:, :, None].astype(np.int64), axis=1)
    rows_v = np.take_along_axis(V, idx[:, :, None].astype(np.int64), axis=1)
    got = orc.insert_rows(np.zeros_like(want), rows_k, rows_v, idx, seeds)
    np.testing.assert_allclose(got, want, rtol=0, atol=0)
    again = orc.insert_rows(got, rows_k, rows_v, idx, seeds)      # additive
    np.testing.assert_allclose(again, 2 * want, rtol=1e-15)


def test_demote_equals_building_the_storage_in_one_go():
    """Compress, append exact tokens, overflow: because insertion is linear and exact rows are
    copies, the storage after the overflow step equals the storage built in one go from all tokens
    with the final retained set."""
    n_inst, N, n_new, D, b, R = 2, 60, 12, 8, 4, 16
    Q = _rand((n_inst, 8, D), 100)
    K, V = _rand((n_inst, N + n_new, D), 101), _rand((n_inst, N + n_new, D), 102)
    seeds = synth.hash_seeds(103)
    c = orc.compress(Q, K[:, :N], V[:, :N], R=R, n_recent=4, seeds=seeds, b=b)
    new_idx = np.arange(N, N + n_new, dtype=np.int32)[None].repeat(n_inst, 0)
    Kr = np.concatenate([c["Kr"], K[:, N:]], axis=1)
    Vr = np.concatenate([c["Vr"], V[:, N:]], axis=1)
    ret = np.concatenate([c["ret_idx"], new_idx], axis=1)
    row_scores = _rand((n_inst, R + n_new), 104) ** 2
    row_scores[0, 3] = row_scores[0, 9]                           # a tie: the older token must win
    keep, evict, cells2 = orc.demote(Kr, Vr, ret, row_scores, c["cells"], R, 4, seeds)
    assert keep.shape == (n_inst, R) and evict.shape == (n_inst, n_new)
    for u in range(n_inst):
        kept_tokens = ret[u][keep[u]]
        assert (np.diff(kept_tokens) > 0).all() and set(kept_tokens[-4:]) == set(range(N + n_new - 4, N + n_new))
        order = np.lexsort((np.arange(R + n_new - 4), -row_scores[u, :R + n_new - 4]))
        assert set(keep[u][:R - 4]) == set(order[:R - 4])
        vague = np.setdiff1d(np.arange(N + n_new), kept_tokens).astype(np.int32)
        want = orc.insert(K[u:u + 1], V[u:u + 1], vague[None], seeds, b)
        np.testing.assert_allclose(cells2[u], want[0], rtol=1e-12, atol=1e-12)


def _swap_case(seed, N=48, D=8, b=4, R=12, n_recent=3, injective=False):
    Q = _rand((1, 8, D), seed)
    K, V = _rand((1, N, D), seed + 1), _rand((1, N, D), seed + 2)
    seeds = synth.injective_seeds() if injective else synth.hash_seeds(seed + 3)
    bb = N if injective else b
    c = orc.compress(Q, K, V, R=R, n_recent=n_recent, seeds=seeds, b=bb, mix=not injective)
    rng = np.random.default_rng(seed + 4)
    tok_scores = rng.random(N).astype(np.float32)              # fresh accumulated scores, all distinct
    row_scores = tok_scores[c["ret_idx"][0]].copy()
    return K, V, seeds, bb, c, tok_scores, row_scores


def test_swap_with_rate_one_leaves_the_top_scores_in_the_candidate_part():
    """ReplaceRate = 1 and no limit: the loop exchanges minimum against maximum until no vague token
    outscores a candidate, so the Candidate part ends as the |C| best-scored tokens of C + V; the
    Recent rows are untouched and the sizes never change."""
    K, V, seeds, b, c, tok, rows = _swap_case(200)
    R, n_recent, N = 12, 3, 48
    Kr, Vr, ret, rs, ts, cells, n = orc.swap(c["Kr"][0], c["Vr"][0], c["ret_idx"][0], rows, tok, c["cells"][0],
                                             n_recent, 1.0, 10 ** 6, seeds)
    assert n > 0
    recent = c["ret_idx"][0][R - n_recent:]
    assert (ret[R - n_recent:] == recent).all() and (Kr[R - n_recent:] == c["Kr"][0][R - n_recent:]).all()
    pool = np.setdiff1d(np.arange(N), recent)
    best = pool[np.argsort(-tok[pool].astype(np.float64), kind="stable")[:R - n_recent]]
    assert set(ret[:R - n_recent]) == set(best)
    assert len(set(ret)) == R
    np.testing.assert_array_equal(rs, tok[ret])                    # scores travel with their tokens
    vague = np.setdiff1d(np.arange(N), ret)
    assert rs[:R - n_recent].min() >= ts[vague].max()              # the loop's exit condition
    np.testing.assert_array_equal(ts[vague], tok[vague])


@pytest.mark.parametrize("seed,rate,limit", [(210, 1.0, 10 ** 6), (211, 1.1, 10 ** 6), (212, 1.5, 7), (213, 1.0, 5),
                                             (214, 1.1, 10 ** 6), (215, 2.0, 10 ** 6)])
def test_swap_loop_pairs_sorted_candidates_with_sorted_vague_tokens(seed, rate, limit):
    """With ReplaceRate >= 1 and scores >= 0 the loop never touches a token twice, so its k-th exchange is
    the k-th worst candidate (score, then token index) against the k-th best vague token (score
    descending, then token index) of the lists as they stand at entry, until the first pair that fails
    C.Min * ReplaceRate < V.Max.  Written out here with two sorts, scores with many ties included, and
    compared with the loop taken one exchange at a time: which rows hold which tokens and scores."""
    K, V, seeds, b, c, tok, rows = _swap_case(seed)
    R, n_recent, N = 12, 3, 48
    rng = np.random.default_rng(seed)
    tok = (rng.integers(0, 6, size=N) / 4.0).astype(np.float32)                # few distinct values: ties everywhere
    rows = (rng.integers(0, 6, size=R) / 4.0).astype(np.float32)
    ret0 = c["ret_idx"][0]
    Kr, Vr, ret, rs, ts, cells, n = orc.swap(c["Kr"][0], c["Vr"][0], ret0, rows, tok, c["cells"][0], n_recent, rate, limit, seeds)
    n_cand = R - n_recent
    cand = sorted(range(n_cand), key=lambda r: (rows[r], ret0[r]))              # rows, worst first
    vague = sorted(np.setdiff1d(np.arange(N), ret0), key=lambda J: (-float(tok[J]), J))     # tokens, best first
    want_ret, want_rs, want_ts = ret0.copy(), rows.copy(), tok.copy()
    k = 0
    while k < min(limit, n_cand, len(vague)):
        r, J = cand[k], vague[k]
        if not (np.float32(rows[r] * np.float32(rate)) < tok[J]):
            break
        want_ts[ret0[r]] = rows[r]
        want_ret[r], want_rs[r] = J, tok[J]
        k += 1
    assert n == k
    np.testing.assert_array_equal(ret, want_ret)
    np.testing.assert_array_equal(rs, want_rs)
    left = np.setdiff1d(np.arange(N), want_ret)
    np.testing.assert_array_equal(ts[left], want_ts[left])


def test_swap_under_injective_hashing_revives_exactly_and_keeps_the_sketch_consistent():
    """One cell per token (no collisions): V.Query returns the original vectors, so a revived row is
    the token's own K, V, and after Delete + Insert the cells equal a sketch built directly from the
    final vague set (linearity of Algorithm 1)."""
    K, V, seeds, b, c, tok, rows = _swap_case(300, injective=True)
    N = 48
    Kr, Vr, ret, rs, ts, cells, n = orc.swap(c["Kr"][0], c["Vr"][0], c["ret_idx"][0], rows, tok, c["cells"][0],
                                             3, 1.1, 10 ** 6, seeds, mix=False)
    assert n > 0
    np.testing.assert_allclose(Kr, K[0][ret], rtol=0, atol=1e-12)
    np.testing.assert_allclose(Vr, V[0][ret], rtol=0, atol=1e-12)
    vague = np.setdiff1d(np.arange(N), ret).astype(np.int32)
    want = orc.insert(K, V, vague[None], seeds, b, mix=False)[0]
    np.testing.assert_allclose(cells, want, rtol=0, atol=1e-12)


def test_swap_rate_and_limit():
    """A swap needs C.Min * ReplaceRate < V.Max: a rate above max/min forbids every swap; max_swaps
    bounds the loop; one swap moves exactly the minimum candidate and the maximum vague token."""
    K, V, seeds, b, c, tok, rows = _swap_case(400)
    args = (c["Kr"][0], c["Vr"][0], c["ret_idx"][0], rows, tok, c["cells"][0], 3)
    out = orc.swap(*args, 1e9, 100, seeds)
    assert out[6] == 0 and (out[2] == c["ret_idx"][0]).all() and np.array_equal(out[5], c["cells"][0])
    out = orc.swap(*args, 1.0, 1, seeds)
    assert out[6] == 1
    cand = c["ret_idx"][0][:9]
    vague = np.setdiff1d(np.arange(48), c["ret_idx"][0])
    j_out, j_in = cand[np.argmin(rows[:9])], vague[np.argmax(tok[vague])]
    changed = np.nonzero(out[2] != c["ret_idx"][0])[0]
    assert len(changed) == 1 and c["ret_idx"][0][changed[0]] == j_out and out[2][changed[0]] == j_in
    # Delete(tmp) then Insert(row): the cells moved by exactly those two contributions
    Kt, Vt = orc.query(c["cells"], np.array([[j_in]], np.int32), seeds)
    step = orc.insert_rows(c["cells"], -Kt, -Vt, np.array([[j_in]], np.int32), seeds)
    step = orc.insert_rows(step, c["Kr"][:, changed], c["Vr"][:, changed], np.array([[j_out]], np.int32), seeds)
    np.testing.assert_allclose(out[5], step[0], rtol=0, atol=1e-12)


def _sdpa_causal_tail(q, K, V, Qn, causal):
    """torch fp64 attention of Qn queries per head over N tokens; with `causal`, query t is token
    N - Qn + t and sees the tokens up to itself (mask written out)."""
    n_inst, G, _, D = q.shape
    N = K.shape[1]
    qt, Kt, Vt = (torch.from_numpy(np.asarray(x, np.float64)) for x in (q, K, V))
    logits = torch.einsum("ugtd,ujd->ugtj", qt, Kt) / np.sqrt(D)
    if causal:
        j = torch.arange(N)[None, :]
        t = torch.arange(Qn)[:, None]
        logits = logits.masked_fill((j > N - Qn + t)[None, None], float("-inf"))
    return torch.einsum("ugtj,ujd->ugtd", torch.softmax(logits, dim=-1), Vt).numpy()


@pytest.mark.parametrize("causal", [True, False])
def test_decode_mq_at_full_budget_is_masked_textbook_attention(causal):
    """Nothing compressed: Qn queries per head against a library softmax attention with the causal
    mask among the queries' own tokens written out."""
    n_inst, G, Qn, N, D = 2, 3, 5, 37, 8
    q = _rand((n_inst, G, Qn, D), 800)
    K, V = _rand((n_inst, N, D), 801), _rand((n_inst, N, D), 802)
    seeds = synth.hash_seeds(803)
    ret = np.arange(N, dtype=np.int32)[None].repeat(n_inst, 0)
    cells = np.zeros((n_inst, 3, 4, 2, D))
    got = orc.decode_mq(q, K, V, ret, cells, N, seeds, causal=causal)
    np.testing.assert_allclose(got, _sdpa_causal_tail(q, K, V, Qn, causal), rtol=1e-10, atol=1e-12)


def test_decode_mq_under_injective_hashing_and_against_single_query_decode():
    """Partial budget with one cell per token: the rebuilt cache is the original one, so the result is
    masked attention over the original K, V; one query per head is `decode`; without the mask every
    query is `decode` over the whole storage; the last query of the causal form sees everything."""
    n_inst, G, Qn, N0, D = 2, 2, 4, 30, 8
    N = N0 + Qn
    q = _rand((n_inst, G, Qn, D), 810)
    K, V = _rand((n_inst, N, D), 811), _rand((n_inst, N, D), 812)
    Qobs = _rand((n_inst, 6, D), 813)
    seeds = synth.injective_seeds()
    c = orc.compress(Qobs, K[:, :N0], V[:, :N0], R=9, n_recent=2, seeds=seeds, b=N, mix=False)
    new = np.arange(N0, N, dtype=np.int32)[None].repeat(n_inst, 0)
    Kr, Vr = np.concatenate([c["Kr"], K[:, N0:]], axis=1), np.concatenate([c["Vr"], V[:, N0:]], axis=1)
    ret = np.concatenate([c["ret_idx"], new], axis=1)
    got = orc.decode_mq(q, Kr, Vr, ret, c["cells"], N, seeds, causal=True, mix=False)
    np.testing.assert_allclose(got, _sdpa_causal_tail(q, K, V, Qn, True), rtol=1e-9, atol=1e-11)
    free = orc.decode_mq(q, Kr, Vr, ret, c["cells"], N, seeds, causal=False, mix=False)
    for t in range(Qn):
        np.testing.assert_allclose(free[:, :, t], orc.decode(q[:, :, t], Kr, Vr, ret, c["cells"], N, seeds, mix=False), rtol=0, atol=0)
    np.testing.assert_allclose(got[:, :, Qn - 1], free[:, :, Qn - 1], rtol=0, atol=0)
    one = orc.decode_mq(q[:, :, :1], Kr, Vr, ret, c["cells"], N, seeds, causal=False, mix=False)
    np.testing.assert_allclose(one[:, :, 0], orc.decode(q[:, :, 0], Kr, Vr, ret, c["cells"], N, seeds, mix=False), rtol=0, atol=0)
    # with collisions (ordinary hashing) the mask still only hides the later queries' tokens
    seeds2 = synth.hash_seeds(814)
    c2 = orc.compress(Qobs, K[:, :N0], V[:, :N0], R=9, n_recent=2, seeds=seeds2, b=3)
    Kr2, Vr2 = np.concatenate([c2["Kr"], K[:, N0:]], axis=1), np.concatenate([c2["Vr"], V[:, N0:]], axis=1)
    ret2 = np.concatenate([c2["ret_idx"], new], axis=1)
    mq = orc.decode_mq(q, Kr2, Vr2, ret2, c2["cells"], N, seeds2, causal=True)
    first = orc.decode(q[:, :, 0], Kr2[:, :9 + 1], Vr2[:, :9 + 1], ret2[:, :9 + 1], c2["cells"], N0 + 1, seeds2)
    np.testing.assert_allclose(mq[:, :, 0], first, rtol=0, atol=0)


def _stream_case(seed, N=40, n_total=64, D=8, b=5, R=14, n_recent=4, injective=False):
    Q = _rand((1, 8, D), seed)
    K, V = _rand((1, n_total, D), seed + 1), _rand((1, n_total, D), seed + 2)
    seeds = synth.injective_seeds() if injective else synth.hash_seeds(seed + 3)
    bb = n_total if injective else b
    c = orc.compress(Q, K[:, :N], V[:, :N], R=R, n_recent=n_recent, seeds=seeds, b=bb, mix=not injective)
    return K, V, seeds, bb, c, c["scores32"][0].copy()         # per-token scores of the N tokens that exist so far


def test_compress_stream_equals_overflow_step_then_swap_loop():
    """Algorithm 3 taken step by step (push, bulk move out of the Recent part, pops of the minimum one
    at a time, swap loop) against the two building blocks pinned above: the pops, for a fixed score
    array, leave the same rows as the top-k rule of `demote` (older token kept among equals), insertion
    is linear so the order of the pops does not matter to the cells, and the swap loop is `swap`."""
    K, V, seeds, b, c, tok = _stream_case(700)
    N, n_new, R, n_recent = 40, 9, 14, 4
    rng = np.random.default_rng(701)
    rows = (rng.random(R) ** 2).astype(np.float32)
    rows[2] = rows[6]                                             # a tie among candidates
    tok = np.concatenate([rng.random(N).astype(np.float32), np.zeros(n_new, np.float32)])   # vague tokens with fresh scores
    tok[c["ret_idx"][0]] = rows
    r_budget, c_budget, slack = 6, 8, 3                           # 4 + 9 = 13 > 6 + 3: the Recent part overflows
    idx_new = np.arange(N, N + n_new, dtype=np.int32)
    got = orc.compress_stream(c["Kr"][0], c["Vr"][0], c["ret_idx"][0], rows, n_recent, tok, c["cells"][0],
                              K[0, N:N + n_new], V[0, N:N + n_new], idx_new, r_budget, c_budget, slack, 1.1, 50, seeds)
    # the same through demote + swap
    Kc = np.concatenate([c["Kr"], K[:, N:N + n_new]], axis=1)
    Vc = np.concatenate([c["Vr"], V[:, N:N + n_new]], axis=1)
    rc = np.concatenate([c["ret_idx"], idx_new[None]], axis=1)
    sc = np.concatenate([rows, np.zeros(n_new, np.float32)])[None]
    n_after, rec_after = orc.append_sizes(R, n_recent, n_new, r_budget, c_budget, slack)
    assert (n_after, rec_after) == (c_budget + r_budget, r_budget)
    keep, evict, cells2 = orc.demote(Kc, Vc, rc, sc, c["cells"], n_after, rec_after, seeds)
    tok2 = tok.copy()
    tok2[rc[0][evict[0]]] = sc[0][evict[0]]
    want = orc.swap(Kc[0][keep[0]], Vc[0][keep[0]], rc[0][keep[0]], sc[0][keep[0]], tok2, cells2[0], rec_after, 1.1, 50, seeds)
    assert got[4] == rec_after and got[7] == want[6] and got[7] > 0
    for a_, b_ in zip(got[:4], want[:4]):
        np.testing.assert_array_equal(a_, b_)
    np.testing.assert_array_equal(got[5], want[4])
    np.testing.assert_allclose(got[6], want[5], rtol=0, atol=1e-11)


def test_compress_stream_slack_holds_the_recent_part_and_sizes_follow_the_counting_rule():
    """Several Slack periods, one or two tokens per call: the Recent part grows until it exceeds its
    budget by more than Slack, then drops to its budget in one go; the Candidate part never exceeds its
    budget; `append_sizes` predicts every size from the counts alone; the retained tokens are distinct
    and the newest tokens are always the Recent rows."""
    K, V, seeds, b, c, tok = _stream_case(710, N=40, n_total=64)
    Kr, Vr, ret, n_recent = c["Kr"][0], c["Vr"][0], c["ret_idx"][0], 4
    rows = tok[ret].copy()
    cells, ctx = c["cells"][0], 40
    r_budget, c_budget, slack = 4, 10, 5
    seen_drop = 0
    rng = np.random.default_rng(711)
    while ctx < 64:
        n_new = min(int(rng.integers(1, 3)), 64 - ctx)
        want_rows, want_recent = orc.append_sizes(len(ret), n_recent, n_new, r_budget, c_budget, slack)
        rows = rows + (rng.random(len(rows)) * 0.1).astype(np.float32)           # scores keep accumulating
        tok = np.concatenate([tok + (rng.random(len(tok)) * 0.1).astype(np.float32), np.zeros(n_new, np.float32)])
        before_recent = n_recent
        Kr, Vr, ret, rows, n_recent, tok, cells, _ = orc.compress_stream(
            Kr, Vr, ret, rows, n_recent, tok, cells, K[0, ctx:ctx + n_new], V[0, ctx:ctx + n_new],
            np.arange(ctx, ctx + n_new, dtype=np.int32), r_budget, c_budget, slack, 1.1, 10, seeds)
        ctx += n_new
        assert (len(ret), n_recent) == (want_rows, want_recent)
        assert n_recent <= r_budget + slack and len(ret) - n_recent <= c_budget
        if n_recent < before_recent + n_new:
            assert before_recent + n_new > r_budget + slack and n_recent == r_budget
            seen_drop += 1
        assert len(set(ret.tolist())) == len(ret)
        assert (ret[len(ret) - n_recent:] == np.arange(ctx - n_recent, ctx)).all()
    assert seen_drop >= 3                                          # at least three Slack periods were run


def test_compress_stream_under_injective_hashing_is_exact():
    """One cell per token: whatever the history of pushes, pops and swaps, every stored row is the
    token's own vectors and the cells equal a sketch built in one go from the final vague set."""
    K, V, seeds, b, c, tok = _stream_case(720, injective=True)
    Kr, Vr, ret, n_recent = c["Kr"][0], c["Vr"][0], c["ret_idx"][0], 4
    rows, cells, ctx = tok[ret].copy(), c["cells"][0], 40
    rng = np.random.default_rng(721)
    swaps = 0
    while ctx < 64:
        n_new = min(3, 64 - ctx)
        tok = np.concatenate([tok + (rng.random(len(tok)) * 0.5).astype(np.float32), np.zeros(n_new, np.float32)])
        rows = rows + (rng.random(len(rows)) * 0.05).astype(np.float32)
        Kr, Vr, ret, rows, n_recent, tok, cells, n = orc.compress_stream(
            Kr, Vr, ret, rows, n_recent, tok, cells, K[0, ctx:ctx + n_new], V[0, ctx:ctx + n_new],
            np.arange(ctx, ctx + n_new, dtype=np.int32), 4, 10, 2, 1.1, 10, seeds, mix=False)
        ctx += n_new
        swaps += n
        np.testing.assert_allclose(Kr, K[0][ret], rtol=0, atol=1e-11)
        np.testing.assert_allclose(Vr, V[0][ret], rtol=0, atol=1e-11)
        vague = np.setdiff1d(np.arange(ctx), ret).astype(np.int32)
        want = orc.insert(K[:, :ctx], V[:, :ctx], vague[None], seeds, b, mix=False)[0]
        np.testing.assert_allclose(cells, want, rtol=0, atol=1e-11)
    assert swaps > 0


def test_window_scores_match_library_softmax_under_the_causal_mask():
    """In-context observation window: row (head g, query t) is token N - W + t and sees keys up to
    itself.  Against a library softmax with the mask written out; every row still sums to one, so the
    scores add up to G * W; the newest token is scored by the last query of each head alone; with W = 1
    the single query is the last token and sees every key, which is the unmasked score."""
    n_inst, G, W, N, D = 2, 3, 5, 23, 8
    Q, K = _rand((n_inst, G * W, D), 500), _rand((n_inst, N, D), 501)
    s = orc.scores(Q, K, window=W)
    tq, tk = torch.from_numpy(Q).double(), torch.from_numpy(K).double()
    logits = tq @ tk.transpose(1, 2) / math.sqrt(D)                              # [n, G*W, N]
    t_of_row = torch.arange(G * W) % W
    visible = torch.arange(N)[None, :] <= (N - W + t_of_row)[:, None]             # [G*W, N]
    P = torch.softmax(logits.masked_fill(~visible[None], float("-inf")), dim=-1)
    np.testing.assert_allclose(s, P.sum(dim=1).numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(s.sum(axis=1), G * W, rtol=1e-12)
    last_rows = [g * W + W - 1 for g in range(G)]
    np.testing.assert_allclose(s[:, N - 1], P[:, last_rows, N - 1].sum(dim=1).numpy(), rtol=1e-12)
    assert np.abs(s - orc.scores(Q, K)).max() > 1e-3                             # the mask matters
    Q1 = _rand((n_inst, G, D), 502)
    np.testing.assert_allclose(orc.scores(Q1, K, window=1), orc.scores(Q1, K), rtol=1e-13)


def test_paper_split_shares():
    """Recent : Candidate : Vague = 0.45 : 0.45 : 0.10 of the budget (hyper-parameter section), at the
    paper's two operating points: 10 % of 2048 and 25 % of 32768."""
    for N, ratio, want_b in ((2048, 0.10, 7), (32768, 0.25, 273)):
        exact, n_recent, b = orc.paper_split(N, ratio)
        total = round(ratio * N)
        assert b == want_b and exact + 3 * b == total
        assert abs(3 * b / total - 0.10) < 0.005
        assert abs(n_recent / total - 0.45) < 0.005 and abs((exact - n_recent) / total - 0.45) < 0.005


def test_layer_budgets_are_proportional_and_add_up():
    """Equal weights give every layer the mean budget; in general the budgets add up to layers x mean,
    are within one row of the proportional share, never exceed the context, and a zero-weight layer
    gets nothing."""
    assert orc.layer_budgets([1.0] * 5, 2048, 0.10) == [205] * 5
    w = [3.0, 1.0, 0.0, 2.0, 2.0]
    bud = orc.layer_budgets(w, 1000, 0.25)
    assert sum(bud) == 5 * 250 and bud[2] == 0
    for l, x in enumerate(w):
        assert abs(bud[l] - 1250 * x / sum(w)) <= 1
    capped = orc.layer_budgets([100.0, 1.0, 1.0], 100, 0.5)       # proportional share of layer 0 = 147 > context
    assert capped[0] == 100 and sum(capped) == 150 and capped[1] == capped[2] == 25


def test_mean_combine_is_the_average_of_the_three_cells_and_exact_without_collisions():
    """The mean combine (not the paper's choice) returns, per element, the average of the token's three
    cells (values times the token's signs): checked against that sum written out with numpy; it is
    linear in the cells, unlike the median; and with one token per cell it returns the token itself."""
    n_inst, N, D, b = 2, 40, 8, 5
    K, V = _rand((n_inst, N, D), 600), _rand((n_inst, N, D), 601)
    seeds = synth.hash_seeds(602)
    idx = np.arange(3, N, dtype=np.int32)[None].repeat(n_inst, 0)
    cells = orc.insert(K, V, idx, seeds, b)
    Kt, Vt = orc.query(cells, idx, seeds, combine="mean")
    bucket, sign = orc.bucket_sign(idx[0], seeds, b)
    for u in range(n_inst):
        wantK = sum(cells[u, i, bucket[i], 0, :] for i in range(3)) / 3.0
        wantV = sum(cells[u, i, bucket[i], 1, :] * sign[i][:, None] for i in range(3)) / 3.0
        np.testing.assert_allclose(Kt[u], wantK, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(Vt[u], wantV, rtol=1e-13, atol=1e-13)
    Km, _ = orc.query(cells, idx, seeds)
    assert np.abs(Km - Kt).max() > 1e-3                                    # it is not the median
    K2, V2 = orc.query(2.5 * cells, idx, seeds, combine="mean")
    np.testing.assert_allclose(K2, 2.5 * Kt, rtol=1e-13)
    inj = synth.injective_seeds()
    cells_inj = orc.insert(K, V, idx, inj, N, mix=False)
    Ki, Vi = orc.query(cells_inj, idx, inj, mix=False, combine="mean")
    np.testing.assert_allclose(Ki, np.take_along_axis(K, idx[:, :, None].astype(np.int64), axis=1), rtol=0, atol=1e-12)
    np.testing.assert_allclose(Vi, np.take_along_axis(V, idx[:, :, None].astype(np.int64), axis=1), rtol=0, atol=1e-12)
    # decode with the mean combine = textbook attention over the cache rebuilt with it
    q = _rand((n_inst, 2, D), 603)
    ret = np.array([[0, 1, 2]] * n_inst, np.int32)
    out = orc.decode(q, K[:, :3], V[:, :3], ret, cells, N, seeds, combine="mean")
    Kfull, Vfull = K.astype(np.float64).copy(), V.astype(np.float64).copy()
    Kfull[:, 3:], Vfull[:, 3:] = Kt, Vt
    p = torch.softmax(torch.from_numpy(q).double() @ torch.from_numpy(Kfull).transpose(1, 2) / math.sqrt(D), dim=-1)
    np.testing.assert_allclose(out, (p @ torch.from_numpy(Vfull)).numpy(), rtol=1e-11, atol=1e-13)
