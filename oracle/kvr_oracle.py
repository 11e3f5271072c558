"""ctypes front end of the CPU oracle (``kvr_oracle.c``).

TEST INFRASTRUCTURE ONLY: the oracle is the checker, not the product.  Only the test-suite, the
smoke check and the benchmark's CPU-baseline leg load this module; the CUDA library and its
Python binding never do, and this module never imports them.

All arrays are numpy, one leading axis over independent head-instances
(batch x layer x kv-head):

    Q     [n_inst, G*W, D] float32   observation queries of the G query heads of that KV head
    K, V  [n_inst, N, D]   float32   (fp16/bf16 values, exactly representable)
    cells [n_inst, r, b, 2, D] float64   slot 0 = key vector, slot 1 = value vector
    seeds [r, 4] uint32   = A, C, A', C' of  h_i(J) = ((A m(J) + C) mod p) mod b,
                            g_i(J) = +1/-1 by the parity of (A' m(J) + C') mod p,  p = 2^31 - 1,
                            m = 32-bit scrambling bijection (mix=True) or the identity (mix=False)
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "kvr_oracle.c")
_LIB = os.path.join(_HERE, "libkvr_oracle.so")

_c_f32 = ctypes.POINTER(ctypes.c_float)
_c_f64 = ctypes.POINTER(ctypes.c_double)
_c_i32 = ctypes.POINTER(ctypes.c_int32)
_c_u32 = ctypes.POINTER(ctypes.c_uint32)
_c_i8 = ctypes.POINTER(ctypes.c_int8)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no FMA contraction) if missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-ffp-contract=off", "-fPIC", "-shared",
               _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.kvro_max_threads.restype = ctypes.c_int32
    return _lib


def _p(a: np.ndarray, ct):
    return a.ctypes.data_as(ct)


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _seeds(seeds):
    s = np.ascontiguousarray(seeds, dtype=np.uint32)
    assert s.ndim == 2 and s.shape[1] == 4
    return s


def max_threads() -> int:
    return int(lib().kvro_max_threads())


def bucket_sign(J, seeds, b: int, mix: bool = True):
    """h_i(J), g_i(J) for every row i: returns (bucket [r, n] int32, sign [r, n] int8)."""
    J = _i32(J).ravel()
    s = _seeds(seeds)
    r, n = s.shape[0], J.size
    bucket = np.empty((r, n), np.int32)
    sign = np.empty((r, n), np.int8)
    lib().kvro_bucket_sign(_p(s, _c_u32), ctypes.c_int32(int(mix)), ctypes.c_int32(r), ctypes.c_int32(b), _p(J, _c_i32),
                           ctypes.c_int64(n), _p(bucket, _c_i32), _p(sign, _c_i8))
    return bucket, sign


def scores(Q, K, scale: float | None = None, window: int | None = None) -> np.ndarray:
    """Importance scores s[j] = sum over observation rows of softmax_j(q.k_j*scale): float64 [n_inst, N].
    window = W: the rows are G heads x W queries that are the last W context tokens themselves, each
    seeing only the keys up to its own position (in-context observation window)."""
    Q, K = _f32(Q), _f32(K)
    n_inst, n_rows, D = Q.shape
    N = K.shape[1]
    assert K.shape == (n_inst, N, D)
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    s = np.empty((n_inst, N), np.float64)
    if window is not None:
        assert n_rows % window == 0
        lib().kvro_scores_window_batch(ctypes.c_int32(n_inst), _p(Q, _c_f32), ctypes.c_int32(n_rows),
                                       ctypes.c_int32(window), _p(K, _c_f32), ctypes.c_int32(N), ctypes.c_int32(D),
                                       ctypes.c_double(scale), _p(s, _c_f64))
        return s
    lib().kvro_scores_batch(ctypes.c_int32(n_inst), _p(Q, _c_f32), ctypes.c_int32(n_rows),
                            _p(K, _c_f32), ctypes.c_int32(N), ctypes.c_int32(D),
                            ctypes.c_double(scale), _p(s, _c_f64))
    return s


def select(s32, R: int, n_recent: int = 0):
    """Retained / compressed index lists (both ascending) from fp32 scores [n_inst, N]."""
    s32 = _f32(s32)
    n_inst, N = s32.shape
    R = min(R, N)
    assert 0 <= n_recent <= R
    ret = np.empty((n_inst, R), np.int32)
    cmp_ = np.empty((n_inst, N - R), np.int32)
    lib().kvro_select_batch(ctypes.c_int32(n_inst), _p(s32, _c_f32), ctypes.c_int32(N),
                            ctypes.c_int32(R), ctypes.c_int32(n_recent), _p(ret, _c_i32),
                            _p(cmp_, _c_i32))
    return ret, cmp_


def insert(K, V, cmp_idx, seeds, b: int, mix: bool = True) -> np.ndarray:
    """Algorithm 1 over the tokens listed in cmp_idx [n_inst, a]; returns fresh cells."""
    K, V, cmp_idx, s = _f32(K), _f32(V), _i32(cmp_idx), _seeds(seeds)
    n_inst, N, D = K.shape
    a = cmp_idx.shape[1]
    r = s.shape[0]
    cells = np.zeros((n_inst, r, b, 2, D), np.float64)
    lib().kvro_insert_batch(ctypes.c_int32(n_inst), _p(cells, _c_f64), _p(s, _c_u32),
                            ctypes.c_int32(int(mix)), ctypes.c_int32(r), ctypes.c_int32(b), ctypes.c_int32(D), _p(K, _c_f32),
                            _p(V, _c_f32), ctypes.c_int32(N), _p(cmp_idx, _c_i32), ctypes.c_int32(a))
    return cells


_COMBINE = {"median": 0, "mean": 1}


def query(cells, idx, seeds, mix: bool = True, combine: str = "median"):
    """Algorithm 2 for the token indices idx [n_inst, a]: (Kt, Vt) float64 [n_inst, a, D].
    combine = "mean" replaces the paper's element-wise Median of the r collected numbers by their mean."""
    cells = np.ascontiguousarray(cells, np.float64)
    idx, s = _i32(idx), _seeds(seeds)
    n_inst, r, b, _, D = cells.shape
    a = idx.shape[1]
    Kt = np.empty((n_inst, a, D), np.float64)
    Vt = np.empty((n_inst, a, D), np.float64)
    if combine != "median":
        lib().kvro_query_c_batch(ctypes.c_int32(n_inst), _p(cells, _c_f64), _p(s, _c_u32),
                                 ctypes.c_int32(int(mix)), ctypes.c_int32(r), ctypes.c_int32(b), ctypes.c_int32(D),
                                 _p(idx, _c_i32), ctypes.c_int32(a), ctypes.c_int32(_COMBINE[combine]),
                                 _p(Kt, _c_f64), _p(Vt, _c_f64))
        return Kt, Vt
    lib().kvro_query_batch(ctypes.c_int32(n_inst), _p(cells, _c_f64), _p(s, _c_u32),
                           ctypes.c_int32(int(mix)), ctypes.c_int32(r), ctypes.c_int32(b), ctypes.c_int32(D), _p(idx, _c_i32),
                           ctypes.c_int32(a), _p(Kt, _c_f64), _p(Vt, _c_f64))
    return Kt, Vt


def decode(q, Kr, Vr, ret_idx, cells, N: int, seeds, scale: float | None = None,
           mix: bool = True, combine: str = "median") -> np.ndarray:
    """Algorithm 4 followed by ordinary attention: out float64 [n_inst, G, D]."""
    q, Kr, Vr, ret_idx, s = _f32(q), _f32(Kr), _f32(Vr), _i32(ret_idx), _seeds(seeds)
    cells = np.ascontiguousarray(cells, np.float64)
    n_inst, G, D = q.shape
    R = ret_idx.shape[1]
    _, r, b, _, _ = cells.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((n_inst, G, D), np.float64)
    if combine != "median":
        lib().kvro_decode_c_batch(ctypes.c_int32(n_inst), _p(q, _c_f32), ctypes.c_int32(G),
                                  _p(cells, _c_f64), _p(s, _c_u32), ctypes.c_int32(int(mix)),
                                  ctypes.c_int32(r), ctypes.c_int32(b), ctypes.c_int32(D), ctypes.c_int32(N), _p(Kr, _c_f32),
                                  _p(Vr, _c_f32), _p(ret_idx, _c_i32), ctypes.c_int32(R), ctypes.c_double(scale),
                                  ctypes.c_int32(_COMBINE[combine]), _p(out, _c_f64))
        return out
    lib().kvro_decode_batch(ctypes.c_int32(n_inst), _p(q, _c_f32), ctypes.c_int32(G),
                            _p(cells, _c_f64), _p(s, _c_u32), ctypes.c_int32(int(mix)),
                            ctypes.c_int32(r), ctypes.c_int32(b),
                            ctypes.c_int32(D), ctypes.c_int32(N), _p(Kr, _c_f32), _p(Vr, _c_f32),
                            _p(ret_idx, _c_i32), ctypes.c_int32(R), ctypes.c_double(scale),
                            _p(out, _c_f64))
    return out


def decode_mq(q, Kr, Vr, ret_idx, cells, N: int, seeds, causal: bool = True, scale: float | None = None,
              mix: bool = True, combine: str = "median") -> np.ndarray:
    """Several queries per head over the same storage (speculative / chunked decoding): the cache is
    rebuilt by Algorithm 4 and every query attends to it as in `decode`.  q [n_inst, G, Qn, D].
    causal: the last Qn rows of the storage are the queries' own tokens (token indices N - Qn .. N - 1,
    in order); query t sees the cache up to and including its own token, i.e. the first
    rows - Qn + t + 1 rows and the first N - Qn + t + 1 tokens.  Not causal: every query sees all of it.
    out float64 [n_inst, G, Qn, D]."""
    q = _f32(q)
    n_inst, G, Qn, D = q.shape
    rows = _i32(ret_idx).shape[1]
    out = np.empty((n_inst, G, Qn, D), np.float64)
    for t in range(Qn):
        cut = Qn - 1 - t if causal else 0
        out[:, :, t] = decode(q[:, :, t], _f32(Kr)[:, :rows - cut], _f32(Vr)[:, :rows - cut], _i32(ret_idx)[:, :rows - cut],
                              cells, N - cut, seeds, scale, mix, combine)
    return out


def decode_mass(q, Kr, Vr, ret_idx, cells, N: int, seeds, scale: float | None = None,
                mix: bool = True) -> np.ndarray:
    """Attention mass of every one of the N tokens in one decode step (sum over the G query heads
    of the softmax probabilities over the rebuilt cache): float64 [n_inst, N]."""
    q, Kr, Vr, ret_idx, s = _f32(q), _f32(Kr), _f32(Vr), _i32(ret_idx), _seeds(seeds)
    cells = np.ascontiguousarray(cells, np.float64)
    n_inst, G, D = q.shape
    R = ret_idx.shape[1]
    _, r, b, _, _ = cells.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    mass = np.empty((n_inst, N), np.float64)
    lib().kvro_decode_mass_batch(ctypes.c_int32(n_inst), _p(q, _c_f32), ctypes.c_int32(G), _p(cells, _c_f64),
                                 _p(s, _c_u32), ctypes.c_int32(int(mix)), ctypes.c_int32(r), ctypes.c_int32(b),
                                 ctypes.c_int32(D), ctypes.c_int32(N), _p(Kr, _c_f32), _p(Vr, _c_f32),
                                 _p(ret_idx, _c_i32), ctypes.c_int32(R), ctypes.c_double(scale), _p(mass, _c_f64))
    return mass


def insert_rows(cells, Krows, Vrows, token_idx, seeds, mix: bool = True) -> np.ndarray:
    """Algorithm 1 for tokens handed over as explicit rows: returns cells + their contribution.
    Krows, Vrows [n_inst, n, D]; token_idx [n_inst, n]."""
    cells = np.array(cells, np.float64, copy=True, order="C")
    Krows, Vrows, token_idx, s = _f32(Krows), _f32(Vrows), _i32(token_idx), _seeds(seeds)
    n_inst, r, b, _, D = cells.shape
    n = token_idx.shape[1]
    for u in range(n_inst):
        lib().kvro_insert_rows(_p(cells[u], _c_f64), _p(s, _c_u32), ctypes.c_int32(int(mix)), ctypes.c_int32(r),
                               ctypes.c_int32(b), ctypes.c_int32(D), _p(Krows[u], _c_f32), _p(Vrows[u], _c_f32),
                               _p(token_idx[u], _c_i32), ctypes.c_int32(n))
    return cells


def demote(Kr, Vr, ret_idx, row_scores, cells, budget: int, n_recent: int, seeds, mix: bool = True):
    """Overflow step of Algorithm 3 on the exact storage.  The rows (ascending token index) hold
    more than `budget` tokens: the newest n_recent stay (Recent part), the budget - n_recent
    highest accumulated scores among the others stay (Candidate part; equal scores: the older
    token stays), every other row is inserted into the sketch (Algorithm 1).  The swap loop of
    Algorithm 3 is not taken: tokens that became vague stay vague.
    Returns (keep_pos [n_inst, budget], evict_pos [n_inst, rows - budget], new cells)."""
    keep, evict = select(row_scores, budget, n_recent)
    Kr, Vr, ret_idx = _f32(Kr), _f32(Vr), _i32(ret_idx)
    ev64 = evict.astype(np.int64)
    Kev = np.take_along_axis(Kr, ev64[:, :, None], axis=1)
    Vev = np.take_along_axis(Vr, ev64[:, :, None], axis=1)
    tok = np.take_along_axis(ret_idx, ev64, axis=1)
    return keep, evict, insert_rows(cells, Kev, Vev, tok, seeds, mix)


def swap(Kr, Vr, ret_idx, row_scores, tok_scores, cells, n_recent: int, replace_rate: float, max_swaps: int,
         seeds, mix: bool = True, round_rows=None):
    """Swap loop of Algorithm 3 on one storage, one exchange at a time in the algorithm's order: while
    the lowest Candidate score times ReplaceRate is below the highest Vague score, query that vague
    token, remove it from the sketch, insert the lowest-scored candidate into the sketch, and give the
    queried vectors the candidate's row.

    The Candidate part is the rows [0, rows - n_recent) (the newest n_recent rows are the Recent part
    and are never touched); the Vague part is every token whose `vague` flag is set, with its score in
    tok_scores.  V.Delete is Algorithm 1 with the negated vectors (insertion is linear); the comparison
    is taken in fp32 like the scores themselves; equal scores: the lower token index is taken (both
    for the minimum and for the maximum).  C.Push stores the queried vectors in the cache's 16-bit
    type: `round_rows` (array -> array) does that rounding; None keeps them as they are.
    Arguments are for ONE head-instance: Kr, Vr [rows, D]; ret_idx [rows]; row_scores [rows] fp32;
    tok_scores [N] fp32 (entries of vague tokens are read, entries of demoted tokens written);
    cells [r, b, 2, D].  Everything is updated on copies, which are returned:
    (Kr, Vr, ret_idx, row_scores, tok_scores, cells, n_swaps)."""
    Kr, Vr = np.array(Kr, np.float64), np.array(Vr, np.float64)
    ret_idx, row_scores = np.array(ret_idx, np.int32), np.array(row_scores, np.float32)
    tok_scores = np.array(tok_scores, np.float32)
    cells = np.array(cells, np.float64, copy=True, order="C")
    N = tok_scores.shape[0]
    vague = np.ones(N, bool)
    vague[ret_idx] = False
    n_cand = ret_idx.shape[0] - n_recent
    rate = np.float32(replace_rate)
    n_swaps = 0
    while n_swaps < max_swaps and n_cand > 0 and vague.any():
        c_order = np.lexsort((ret_idx[:n_cand], row_scores[:n_cand]))          # score asc, then token index asc
        row = int(c_order[0])
        v_tok = np.nonzero(vague)[0]
        v_order = np.lexsort((v_tok, -tok_scores[v_tok].astype(np.float64)))    # score desc, then token index asc
        J = int(v_tok[v_order[0]])
        c_min, v_max = row_scores[row], tok_scores[J]
        if not (np.float32(c_min * rate) < v_max):
            break
        Kt, Vt = query(cells[None], np.array([[J]], np.int32), seeds, mix)      # tmp <- V.Query(J)
        Kt, Vt = Kt[0, 0], Vt[0, 0]
        one = np.array([[J]], np.int32)
        cells = insert_rows(cells[None], -Kt[None, None], -Vt[None, None], one, seeds, mix)[0]     # remove the queried token from the sketch
        Jc = int(ret_idx[row])
        cells = insert_rows(cells[None], Kr[row][None, None], Vr[row][None, None],
                            np.array([[Jc]], np.int32), seeds, mix)[0]          # the candidate goes into the sketch
        tok_scores[Jc] = c_min
        vague[Jc], vague[J] = True, False
        Kr[row] = round_rows(Kt) if round_rows is not None else Kt               # C.Push(tmp)
        Vr[row] = round_rows(Vt) if round_rows is not None else Vt
        ret_idx[row], row_scores[row] = J, v_max
        n_swaps += 1
    return Kr, Vr, ret_idx, row_scores, tok_scores, cells, n_swaps


def append_sizes(n_rows: int, n_recent: int, n_new: int, r_budget: int, c_budget: int, slack: int):
    """Sizes after Algorithm 3 has taken n_new tokens (counting only; no data is looked at): returns
    (rows_after, recent_after).  The Recent part gives up its oldest tokens only once it exceeds its
    budget by more than Slack, and then all of its excess at once; the Candidate part never keeps more
    than its budget."""
    recent = n_recent + n_new
    cand = n_rows - n_recent
    if recent > r_budget + slack:
        cand += recent - r_budget
        recent = r_budget
    return min(cand, c_budget) + recent, recent


def compress_stream(Kr, Vr, ret_idx, row_scores, n_recent: int, tok_scores, cells, K_new, V_new, idx_new,
                    r_budget: int, c_budget: int, slack: int, replace_rate: float, max_swaps: int,
                    seeds, mix: bool = True, round_rows=None):
    """Algorithm 3 (insert newly generated tokens and compress) for ONE head-instance, in the
    algorithm's order:
      1. the new tokens are pushed to the Recent part (a queue, oldest first; they arrive with score 0);
      2. if the Recent part now exceeds its budget by more than Slack, its oldest tokens, all that
         exceed the budget, move to the Candidate part in one go;
      3. while the Candidate part is over its budget, its lowest-scored token is taken out and inserted
         into the sketch (Algorithm 1); among equal scores the newest goes first, so that the older
         token stays (the same rule as `demote`); the token's score moves to the per-token array;
      4. the swap loop (`swap`).
    The storage is the exact rows in order: Candidate rows first, then the n_recent Recent rows.
    Arguments as in `swap`, plus K_new, V_new [n_new, D] and their token indices idx_new [n_new].
    Everything is updated on copies; returns
    (Kr, Vr, ret_idx, row_scores, n_recent, tok_scores, cells, n_swaps)."""
    Kr, Vr = np.array(Kr, np.float64), np.array(Vr, np.float64)
    ret_idx, row_scores = np.array(ret_idx, np.int32), np.array(row_scores, np.float32)
    tok_scores = np.array(tok_scores, np.float32)
    cells = np.array(cells, np.float64, copy=True, order="C")
    K_new, V_new = np.array(K_new, np.float64), np.array(V_new, np.float64)
    rows = [dict(k=Kr[i], v=Vr[i], idx=int(ret_idx[i]), score=np.float32(row_scores[i])) for i in range(len(ret_idx))]
    cut = len(rows) - n_recent
    C, R = rows[:cut], rows[cut:]
    for j in range(len(idx_new)):                                                # 1. R.Push(T)
        R.append(dict(k=K_new[j], v=V_new[j], idx=int(idx_new[j]), score=np.float32(0.0)))
    if len(R) > r_budget + slack:                                                # 2. R over budget + Slack
        k = len(R) - r_budget
        C.extend(R[:k])
        R = R[k:]
    while len(C) > c_budget:                                                     # 3. pop the minimum into the sketch
        lo = min(range(len(C)), key=lambda i: (C[i]["score"], -i))
        t = C.pop(lo)
        one = np.array([[t["idx"]]], np.int32)
        cells = insert_rows(cells[None], t["k"][None, None], t["v"][None, None], one, seeds, mix)[0]
        tok_scores[t["idx"]] = t["score"]
    rows = C + R
    D = Kr.shape[1] if Kr.ndim == 2 else K_new.shape[1]
    Kr2 = np.array([t["k"] for t in rows], np.float64).reshape(len(rows), D)
    Vr2 = np.array([t["v"] for t in rows], np.float64).reshape(len(rows), D)
    ret2 = np.array([t["idx"] for t in rows], np.int32)
    sc2 = np.array([t["score"] for t in rows], np.float32)
    Kr2, Vr2, ret2, sc2, tok_scores, cells, n = swap(Kr2, Vr2, ret2, sc2, tok_scores, cells, len(R), replace_rate,
                                                      max_swaps, seeds, mix, round_rows)        # 4. swap loop
    return Kr2, Vr2, ret2, sc2, len(R), tok_scores, cells, n


def paper_split(context: int, ratio: float, r: int = 3):
    """Storage split of the paper's hyper-parameter section: Recent 0.45, Candidate 0.45, Vague 0.10 of
    the budget, r = 3 rows, the width b fixed by the Vague share once r is set; one cell counts like one
    token.  Returns (exact_rows, n_recent, b) with exact_rows = Recent + Candidate."""
    total = int(np.floor(ratio * context + 0.5))
    b = max(1, int(np.floor(0.1 * total / r + 0.5)))
    exact = max(0, total - r * b)
    return exact, exact // 2, b


def layer_budgets(weights, context: int, ratio: float):
    """Per-layer budgets proportional to per-layer weights (appendix on Fisher information: the
    weight of a layer "is used to determine the memory budget allocation ratio across different
    layers"; no formula is printed).  Mean budget = floor(ratio * context + 0.5); no layer gets more
    than `context` rows (excess re-shared in proportion); largest remainder settles the fractions,
    the lower layer first among equals."""
    w = [float(x) for x in weights]
    L = len(w)
    total = int(np.floor(ratio * context + 0.5)) * L
    full = [False] * L
    share = [0.0] * L
    left, wleft = float(total), sum(w)
    for _ in range(L):
        capped = False
        for l in range(L):
            if not full[l] and wleft > 0 and left * w[l] / wleft > context:
                full[l], share[l], capped = True, float(context), True
        if not capped:
            break
        left = max(0.0, float(total) - context * sum(full))
        wleft = sum(w[l] for l in range(L) if not full[l])
    for l in range(L):
        if not full[l]:
            share[l] = left * w[l] / wleft if wleft > 0 else 0.0
    budgets = [int(np.floor(s)) for s in share]
    target = min(total, L * context)
    while sum(budgets) < target:
        cand = [(share[l] - np.floor(share[l]), -l) for l in range(L) if budgets[l] < context]
        if not cand:
            break
        l = -max(cand)[1]
        budgets[l] += 1
        share[l] = float(np.floor(share[l]))
    return budgets


def gather(X, ret_idx) -> np.ndarray:
    """Exact rows of the retained tokens: X [n_inst, N, D] -> [n_inst, R, D]."""
    X = _f32(X)
    return np.take_along_axis(X, _i32(ret_idx)[:, :, None].astype(np.int64), axis=1)


def compress(Q, K, V, R: int, n_recent: int, seeds, b: int, scale: float | None = None,
             forced_ret_idx=None, mix: bool = True):
    """One-shot Algorithm 3: scores -> selection -> exact copies + Algorithm 1 for the rest.

    forced_ret_idx (ascending, [n_inst, R]) replaces the selection (used when several selections
    are valid, i.e. scores tie to within floating-point rounding).
    Returns dict(scores64, scores32, ret_idx, cmp_idx, Kr, Vr, cells).
    """
    K = _f32(K)
    n_inst, N, D = K.shape
    s64 = scores(Q, K, scale)
    s32 = s64.astype(np.float32)
    if forced_ret_idx is None:
        ret, cmp_ = select(s32, R, n_recent)
    else:
        ret = _i32(forced_ret_idx)
        mask = np.ones((n_inst, N), bool)
        np.put_along_axis(mask, ret.astype(np.int64), False, axis=1)
        cmp_ = np.stack([np.nonzero(m)[0] for m in mask]).astype(np.int32) if N > ret.shape[1] \
            else np.empty((n_inst, 0), np.int32)
    cells = insert(K, V, cmp_, seeds, b, mix)
    return dict(scores64=s64, scores32=s32, ret_idx=ret, cmp_idx=cmp_, Kr=gather(K, ret),
                Vr=gather(V, ret), cells=cells)
