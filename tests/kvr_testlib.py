"""Shared helpers of the GPU parity tests: run one case through the C ABI (via the Python
binding) and through the CPU oracle on the same seeded inputs, and compare stage by stage.

Comparison protocol
  * integer results are bit-exact: the selection equals the oracle's selection rule applied to the
    scores the kernel stored (the decision is taken in the kernel's precision, fp32, on both
    sides); compressed indices, buckets and signs equal the oracle's; retained rows are exact copies.
  * against the oracle's own (fp64) scores the selection may differ only inside a narrow band around
    the R-th score, where fp32 rounding of nearly tied scores decides: every token clearly above
    the band is kept, none clearly below it.
  * later stages are compared with the oracle re-run on the selection the kernel made.
  * floating-point results: max-abs <= 2e-3 (cells, reconstructed K/V, attention outputs).
"""
from __future__ import annotations

import numpy as np
import torch

import paper_2512_17917_b200 as kvr
from oracle import kvr_oracle as orc
from paper_2512_17917_b200 import synth

TOL = 2e-3          # max-abs bar for cells, reconstructed K/V and attention outputs
SCORE_RTOL = 2e-4   # fp32 tensor-core logits + exp2 vs fp64
BAND = 1e-4         # relative half-width of the selection ambiguity band


def inst_major(x: torch.Tensor) -> np.ndarray:
    """K / V style tensors [..., H, n, D] -> [n_inst, n, D] float32."""
    x = x.detach().cpu().float()
    return x.reshape(-1, x.shape[-2], x.shape[-1]).numpy()


def obs_to_inst(Qobs: torch.Tensor, H: int) -> np.ndarray:
    Q = Qobs.detach().cpu().float()
    Hq, W, D = Q.shape[-3:]
    G = Hq // H
    return Q.reshape(-1, H, G, W, D).reshape(-1, G * W, D).numpy()


def dec_to_inst(q: torch.Tensor, H: int) -> np.ndarray:
    x = q.detach().cpu().float()
    Hq, D = x.shape[-2:]
    G = Hq // H
    return x.reshape(-1, H, G, D).reshape(-1, G, D).numpy()


def make_case(seed, B, H, Hq, N, W, dtype, L=1, n_outlier=4):
    """CPU tensors of L layers: K, V [L,B,H,N,D], Qobs [L,B,Hq,W,D], q [L,B,Hq,D]."""
    Ks, Vs, Qs, qs = [], [], [], []
    for layer in range(L):
        K, V = synth.make_kv(seed + 101 * layer, B, H, N, 128, dtype, "cpu", n_outlier=n_outlier)
        Ks.append(K)
        Vs.append(V)
        Qs.append(synth.make_queries(seed + 101 * layer + 1, B, Hq, W, 128, dtype, "cpu"))
        qs.append(synth.make_decode_q(seed + 101 * layer + 2, B, Hq, 128, dtype, "cpu"))
    return torch.stack(Ks), torch.stack(Vs), torch.stack(Qs), torch.stack(qs)


def sampled_instances(n_inst: int, k: int, salt: int = 0):
    """k head-instances for the oracle to check at full size.  The choice is a fixed function of
    KVR_TEST_SEED (default 0): another seed checks other instances."""
    import os
    rng = np.random.default_rng([int(os.environ.get("KVR_TEST_SEED", "0")), salt, n_inst])
    return sorted(int(x) for x in rng.choice(n_inst, size=min(k, n_inst), replace=False))


def check_selection_band(s64: np.ndarray, ret: np.ndarray, R: int, n_recent: int):
    """Selection vs the oracle's fp64 scores: exact outside the ambiguity band."""
    n_inst, N = s64.shape
    k = R - n_recent
    n_cand = N - n_recent
    for u in range(n_inst):
        kept = np.zeros(N, bool)
        kept[ret[u]] = True
        assert kept.sum() == R
        assert kept[n_cand:].all(), "recent tokens must be kept"
        if k <= 0 or k >= n_cand:
            continue
        c = s64[u, :n_cand]
        thr = np.sort(c)[::-1][k - 1]                 # R-th score
        must = c > thr * (1 + BAND)
        mustnt = c < thr * (1 - BAND)
        assert kept[:n_cand][must].all(), "a clearly higher-scored token was dropped"
        assert not kept[:n_cand][mustnt].any(), "a clearly lower-scored token was kept"


def run_and_check(K, V, Qobs, q, *, R, n_recent, b, seeds, index_mix=True, layer_mode="per_layer",
                  sample_inst=None, check_reconstruct=True, scale=0.0, decode_kernel=None, score_kernel=None, obs_causal=False, combine="median",
                  expect_decode_kernel=None):
    """Compress + one decode step on the GPU through the C ABI, the same through the oracle,
    compare every stage.  K, V, Qobs, q carry a leading layer axis.  Returns (gpu_out, oracle_out)."""
    L, B, H, N, D = K.shape
    Hq, W = Qobs.shape[2], Qobs.shape[3]
    G = Hq // H
    r = int(np.asarray(seeds).shape[0])                      # sketch rows = sets of (A, C, A', C')
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N, r=r,
                               kv_dtype=K.dtype, hash_seeds=seeds, index_mix=index_mix, device=dev)
    if decode_kernel is not None:
        kvr.kvr_sketch_set_decode_kernel(sk, decode_kernel)
    if score_kernel is not None:
        kvr.kvr_sketch_set_score_kernel(sk, score_kernel)
    if obs_causal:
        kvr.kvr_sketch_set_obs_window_causal(sk, True)
    if combine == "mean":
        kvr.kvr_sketch_set_combine(sk, kvr.KVR_COMBINE_MEAN)
    Kd, Vd, Qd, qd = K.to(dev), V.to(dev), Qobs.to(dev), q.to(dev)
    Rr = min(R, N)
    if layer_mode == "all":
        Kr, Vr, ret = kvr.kvr_compress(sk, kvr.KVR_ALL_LAYERS, Kd, Vd, Qd, R, n_recent)
        out = kvr.kvr_decode_attention(sk, kvr.KVR_ALL_LAYERS, qd, Kr, Vr, ret, softmax_scale=scale)
    else:
        Krs, Vrs, rets, outs = [], [], [], []
        for layer in range(L):
            a_, b_, c_ = kvr.kvr_compress(sk, layer, Kd[layer], Vd[layer], Qd[layer], R, n_recent)
            Krs.append(a_), Vrs.append(b_), rets.append(c_)
        for layer in range(L):
            outs.append(kvr.kvr_decode_attention(sk, layer, qd[layer], Krs[layer], Vrs[layer], rets[layer],
                                                 softmax_scale=scale))
        Kr, Vr, ret, out = torch.stack(Krs), torch.stack(Vrs), torch.stack(rets), torch.stack(outs)
    if decode_kernel is not None and decode_kernel != kvr.KVR_DECODE_AUTO:
        assert kvr.kvr_last_decode_kernel(sk) == decode_kernel, "the requested decode kernel did not run"
    if expect_decode_kernel is not None:
        assert kvr.kvr_last_decode_kernel(sk) == expect_decode_kernel, "the library chose another decode kernel"
    if score_kernel is not None and score_kernel != kvr.KVR_SCORE_AUTO:
        assert kvr.kvr_last_score_kernel(sk) == score_kernel, "the requested scoring kernel did not run"
    assert kvr.kvr_sketch_device_status(sk) == 0, "a bounded wait inside a kernel gave up"
    s_gpu = kvr.kvr_get_scores(sk, kvr.KVR_ALL_LAYERS)
    cmp_gpu, bucket_gpu, sign_gpu = kvr.kvr_get_assignment(sk, kvr.KVR_ALL_LAYERS)
    cells_gpu = kvr.kvr_get_cells(sk, kvr.KVR_ALL_LAYERS)
    Kt_gpu, Vt_gpu = kvr.kvr_reconstruct(sk, kvr.KVR_ALL_LAYERS) if check_reconstruct else (None, None)
    torch.cuda.synchronize()

    n_inst = L * B * H
    a = N - Rr
    sel = np.arange(n_inst) if sample_inst is None else np.asarray(sample_inst)
    Kc, Vc = inst_major(K)[sel], inst_major(V)[sel]
    Qc, qc = obs_to_inst(Qobs, H)[sel], dec_to_inst(q, H)[sel]
    s_g = s_gpu.reshape(n_inst, N).cpu().numpy()[sel]
    ret_g = ret.reshape(n_inst, Rr).cpu().numpy()[sel]
    cmp_g = cmp_gpu.reshape(n_inst, a).cpu().numpy()[sel]

    # --- scores -------------------------------------------------------------------------------
    s64 = orc.scores(Qc, Kc, window=W if obs_causal else None)
    np.testing.assert_allclose(s_g, s64, rtol=SCORE_RTOL, atol=1e-7)
    # --- selection: the rule applied to the kernel's own fp32 scores, bit-exact ------------------
    ret_o, cmp_o = orc.select(s_g, Rr, n_recent)
    assert (ret_g == ret_o).all(), "selection differs from the rule applied to the stored scores"
    assert (cmp_g == cmp_o).all()
    check_selection_band(s64, ret_g, Rr, n_recent)
    # --- exact copies --------------------------------------------------------------------------
    Kr_g = inst_major(Kr)[sel] if Rr else np.zeros((len(sel), 0, D), np.float32)
    Vr_g = inst_major(Vr)[sel] if Rr else np.zeros((len(sel), 0, D), np.float32)
    assert (Kr_g == orc.gather(Kc, ret_g)).all() and (Vr_g == orc.gather(Vc, ret_g)).all()
    # --- hashing -------------------------------------------------------------------------------
    if a:
        bk = bucket_gpu.reshape(n_inst, r, a).cpu().numpy()[sel]
        sg = sign_gpu.reshape(n_inst, r, a).cpu().numpy()[sel]
        for u in range(len(sel)):
            bo, so = orc.bucket_sign(cmp_g[u], seeds, b, mix=index_mix)
            assert (bk[u] == bo).all() and (sg[u] == so).all(), "bucket / sign assignment"
    # --- cells (oracle re-run on the kernel's selection) -----------------------------------------
    cells_o = orc.insert(Kc, Vc, cmp_g, seeds, b, mix=index_mix)              # [n, r, b, 2, D]
    cells_g = cells_gpu.reshape(n_inst, 2, r, b, D).cpu().numpy()[sel].transpose(0, 2, 3, 1, 4)
    assert np.abs(cells_g - cells_o).max() <= TOL, np.abs(cells_g - cells_o).max()
    # --- reconstruction ------------------------------------------------------------------------
    if check_reconstruct and a:
        Kt_o, Vt_o = orc.query(cells_o, cmp_g, seeds, mix=index_mix, combine=combine)
        dk = np.abs(Kt_gpu.reshape(n_inst, a, D).cpu().numpy()[sel] - Kt_o).max()
        dv = np.abs(Vt_gpu.reshape(n_inst, a, D).cpu().numpy()[sel] - Vt_o).max()
        assert dk <= TOL and dv <= TOL, (dk, dv)
    # --- decode attention ------------------------------------------------------------------------
    out_o = orc.decode(qc, Kr_g, Vr_g, ret_g, cells_o, N, seeds, scale=(scale or None), mix=index_mix, combine=combine)
    out_g = out.reshape(n_inst, G, D).cpu().numpy()[sel]
    err = np.abs(out_g - out_o).max()
    assert np.isfinite(out_g).all() and err <= TOL, err
    kvr.kvr_sketch_destroy(sk)
    return out_g, out_o


def run_stream_case(*, which, dtype, one_call, B, H, Hq, N, R, b, n_rec0, r_budget, c_budget, slack, steps, rate, max_swaps,
                    seed):
    """A generation loop on the GPU (decode, score accumulation, kvr_append per step) against the oracle's
    compress_stream, every step and every head-instance.  one_call: the decode call keeps the step's scores
    (kvr_decode_attention_scored) instead of two accumulate calls after it.  Returns (steps in which the
    Recent part overflowed, swaps in total)."""
    G = Hq // H
    n_inst = B * H
    seeds = synth.hash_seeds(seed)
    total = N + sum(steps)
    K, V, Q, q = make_case(seed + 1, B, H, Hq, total, 8, dtype, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=total, kv_dtype=dtype,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
    Kall, Vall = inst_major(K[0]), inst_major(V[0])
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0, :, :, :N].contiguous().to(dev), V[0, :, :, :N].contiguous().to(dev),
                                   Q[0].to(dev), R, n_rec0)
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(n_inst, -1).cpu().numpy()
    s0 = kvr.kvr_get_scores(sk, 0).reshape(n_inst, -1)
    acc = torch.gather(s0, 1, ret.reshape(n_inst, -1).long()).reshape(B, H, min(R, N)).contiguous()
    # oracle state per head-instance
    o_cells = list(orc.insert(Kall[:, :N], Vall[:, :N], cmp0, seeds, b))
    o_Kr, o_Vr = list(inst_major(Kr).astype(np.float64)), list(inst_major(Vr).astype(np.float64))
    o_ret = list(ret.reshape(n_inst, -1).cpu().numpy())
    n_recent, ctx, drops, swaps = n_rec0, N, 0, 0
    rounder = lambda x: torch.from_numpy(np.asarray(x, np.float64)).to(dtype).double().numpy()
    ulp = 2.0 ** -11 if dtype == torch.float16 else 2.0 ** -8
    for it, n_new in enumerate(steps):
        # ---- decode over the current storage, then the attention mass goes to the scores
        qd = synth.make_decode_q(seed + 300 + it, B, Hq, 128, dtype, dev)
        if one_call:
            out = kvr.kvr_decode_attention_scored(sk, 0, qd, Kr, Vr, ret, acc)
        else:
            out = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
            kvr.kvr_accumulate_scores(sk, 0, qd, Kr, acc)
            kvr.kvr_accumulate_vague_scores(sk, 0, qd)
        qo = dec_to_inst(qd, H)
        want = orc.decode(qo, np.stack(o_Kr), np.stack(o_Vr), np.stack(o_ret), np.stack(o_cells), ctx, seeds)
        assert np.abs(out.reshape(n_inst, G, 128).cpu().numpy() - want).max() <= TOL
        tok_g = kvr.kvr_get_scores(sk, 0).reshape(n_inst, -1).cpu().numpy()       # [n_inst, context of the last overflow step]
        acc_np = acc.reshape(n_inst, -1).cpu().numpy()
        # ---- Algorithm 3 for the new tokens
        Kn, Vn = K[0, :, :, ctx:ctx + n_new].contiguous().to(dev), V[0, :, :, ctx:ctx + n_new].contiguous().to(dev)
        before = n_recent + n_new
        Kr, Vr, ret, acc, n_recent_g, n_sw = kvr.kvr_append(sk, 0, Kr, Vr, ret, acc, n_recent, Kn, Vn, r_budget, c_budget,
                                                            slack, rate, max_swaps)
        assert kvr.kvr_sketch_device_status(sk) == 0
        n_sw = n_sw.reshape(n_inst).cpu().numpy()
        ret_g, acc_g = ret.reshape(n_inst, -1).cpu().numpy(), acc.reshape(n_inst, -1).cpu().numpy()
        cells_g = kvr.kvr_get_cells(sk, 0).reshape(n_inst, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4)
        tok_after = kvr.kvr_get_scores(sk, 0).reshape(n_inst, -1).cpu().numpy()
        for u in range(n_inst):
            # the oracle steps from its own storage, with the scores the kernels accumulated
            tok_u = np.concatenate([tok_g[u], np.zeros(ctx + n_new - tok_g.shape[1], np.float32)])   # tokens beyond are rows
            Ko, Vo, ro, so, rec_o, to, co, n = orc.compress_stream(
                o_Kr[u], o_Vr[u], o_ret[u], acc_np[u], n_recent, tok_u, o_cells[u], Kall[u, ctx:ctx + n_new],
                Vall[u, ctx:ctx + n_new], np.arange(ctx, ctx + n_new, dtype=np.int32), r_budget, c_budget, slack, rate,
                max_swaps, seeds, round_rows=rounder)
            assert rec_o == n_recent_g and n == n_sw[u]
            assert (ret_g[u] == ro).all() and (acc_g[u] == so).all()
            vague = np.setdiff1d(np.arange(ctx + n_new), ro)
            assert (tok_after[u, vague] == to[vague]).all()
            # (the tolerance is derived for cells up to about 500 in magnitude and a few updates per cell; a sketch
            # of a handful of cells sums thousands of tokens per cell, and every swap rounds the cells it touches
            # to fp32 again, a random walk of half-units in the last place: the bar grows with both)
            cmax = float(np.abs(co).max())
            tol = TOL * max(1.0, cmax / 500.0) + np.sqrt(swaps + n + 1.0) * 2.0 ** -22 * cmax
            err = float(np.abs(cells_g[u] - co).max())
            assert err <= tol, (err, tol)
            dk, dv = np.abs(inst_major(Kr)[u] - Ko), np.abs(inst_major(Vr)[u] - Vo)
            assert (dk <= tol + 2 * ulp * np.abs(Ko)).all() and (dv <= tol + 2 * ulp * np.abs(Vo)).all()
            # carry the GPU's rows on (a revived row is rounded to the cache type on both sides)
            o_Kr[u], o_Vr[u], o_ret[u], o_cells[u] = inst_major(Kr)[u].astype(np.float64), inst_major(Vr)[u].astype(np.float64), ro, co
            swaps += n
        drops += int(n_recent_g < before)
        n_recent, ctx = n_recent_g, ctx + n_new
    # ---- one more decode over the final storage
    qd = synth.make_decode_q(seed + 999, B, Hq, 128, dtype, dev)
    out = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
    want = orc.decode(dec_to_inst(qd, H), np.stack(o_Kr), np.stack(o_Vr), np.stack(o_ret), np.stack(o_cells), ctx, seeds)
    assert np.abs(out.reshape(n_inst, G, 128).cpu().numpy() - want).max() <= TOL
    kvr.kvr_sketch_destroy(sk)
    return drops, swaps
