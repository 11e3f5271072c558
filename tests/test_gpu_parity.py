"""GPU parity tests: the CUDA path, called through the C ABI, against the CPU oracle on the same
seeded inputs, element by element (protocol and tolerances in kvr_testlib)."""
import math

import numpy as np
import pytest
import torch

import paper_2512_17917_b200 as kvr
from oracle import kvr_oracle as orc
from paper_2512_17917_b200 import synth

from kvr_testlib import TOL, dec_to_inst, inst_major, make_case, obs_to_inst, run_and_check, run_stream_case, sampled_instances

pytestmark = pytest.mark.gpu
F16, BF16 = torch.float16, torch.bfloat16


@pytest.mark.parametrize("B,H,Hq,L,N,W,R,n_recent,b,dtype,mode", [
    (2, 2, 8, 2, 333, 5, 40, 7, 5, F16, "per_layer"),      # several key tiles, ragged tail, Recent part
    (1, 2, 8, 1, 1000, 32, 100, 0, 4, BF16, "per_layer"),   # bf16, full 128-row observation tile
    (1, 2, 8, 3, 777, 32, 194, 97, 9, F16, "all"),          # all layers in one launch, paper's Recent/Candidate split
    (1, 2, 2, 1, 200, 3, 20, 0, 3, F16, "per_layer"),       # G = 1 (no GQA, the paper's Llama-2 case)
    (1, 1, 8, 1, 130, 40, 13, 0, 2, F16, "per_layer"),      # G = 8, W = 40: 320 observation rows = 3 row tiles
    (1, 3, 6, 1, 257, 7, 26, 2, 300, BF16, "per_layer"),    # G = 2, more cells than tokens
    (1, 1, 4, 1, 2100, 32, 210, 0, 7, F16, "per_layer"),    # more than 2048 tokens: three selection tiles
])
def test_small_cases(B, H, Hq, L, N, W, R, n_recent, b, dtype, mode):
    K, V, Q, q = make_case(100 + N, B, H, Hq, N, W, dtype, L)
    run_and_check(K, V, Q, q, R=R, n_recent=n_recent, b=b, seeds=synth.hash_seeds(N), layer_mode=mode)


@pytest.mark.parametrize("B,H,Hq,L,N,W,R,n_recent,b,dtype,mode", [
    (1, 2, 8, 1, 700, 4, 70, 3, 5, F16, "per_layer"),       # one class, a few tokens per half-warp, ragged last round
    (2, 2, 8, 2, 3000, 8, 300, 0, 37, BF16, "all"),         # bf16, all layers in one launch
    (1, 2, 4, 1, 1500, 4, 150, 10, 300, F16, "per_layer"),  # G = 2, more cells than tokens per bucket (empty buckets)
    (1, 3, 3, 1, 900, 4, 0, 0, 11, F16, "per_layer"),       # G = 1, nothing retained
    (1, 1, 4, 1, 9000, 8, 900, 0, 64, F16, "per_layer"),
    (1, 2, 8, 1, 6000, 8, 1500, 0, 200, F16, "per_layer"),   # 4 x 4 classes (wide sketch), several row-0 runs per half-warp
    (1, 1, 4, 1, 4000, 8, 400, 0, 500, BF16, "per_layer"),    # 8 x 8 classes, mostly empty row-0 cells    # one head-instance, class lists cut into many slices
    (1, 2, 8, 1, 300, 4, 290, 0, 4, F16, "per_layer"),      # fewer compressed tokens than token groups
])
def test_staged_kernel_small_cases(B, H, Hq, L, N, W, R, n_recent, b, dtype, mode):
    """The staged decode kernel (tokens grouped into classes whose rows-1-and-2 cells sit in shared
    memory), forced on sizes the library might hand to the split kernel, against the oracle."""
    K, V, Q, q = make_case(900 + N, B, H, Hq, N, W, dtype, L)
    run_and_check(K, V, Q, q, R=R, n_recent=n_recent, b=b, seeds=synth.hash_seeds(N + 7), layer_mode=mode,
                  decode_kernel=kvr.KVR_DECODE_STAGED)


@pytest.mark.parametrize("B,H,Hq,L,N,W,R,b,dtype,mode", [
    (1, 2, 8, 1, 1000, 32, 100, 4, BF16, "per_layer"),   # one full 128-row tile of observation rows, ragged key tail
    (1, 1, 8, 1, 130, 40, 13, 2, F16, "per_layer"),      # 320 observation rows = three row tiles; 2 keys in the last key tile
    (2, 2, 4, 1, 640, 24, 64, 5, F16, "per_layer"),      # 48 rows per head-instance: a row tile reaches into the next instance
    (1, 4, 16, 2, 4099, 32, 400, 30, F16, "all"),        # several key chunks per head-instance, all layers in one call
    (1, 2, 8, 1, 128, 32, 128, 1, F16, "per_layer"),     # exactly one key tile, everything retained
])
@pytest.mark.parametrize("score_kernel", ["tcgen05", "mma_sync"])
def test_scoring_kernels(B, H, Hq, L, N, W, R, b, dtype, mode, score_kernel):
    """Both importance-scoring kernels (tcgen05 + tensor memory + TMA; mma.sync), each forced, against
    the oracle through the whole path."""
    which = kvr.KVR_SCORE_TCGEN05 if score_kernel == "tcgen05" else kvr.KVR_SCORE_MMA_SYNC
    K, V, Q, q = make_case(300 + N, B, H, Hq, N, W, dtype, L)
    run_and_check(K, V, Q, q, R=R, n_recent=0, b=b, seeds=synth.hash_seeds(N + 1), layer_mode=mode,
                  score_kernel=which)


@pytest.mark.parametrize("B,H,Hq,N,W,R,b,dtype", [
    (1, 2, 8, 1000, 32, 100, 4, F16),      # the window spans the ragged last key tile
    (2, 2, 4, 640, 24, 64, 5, BF16),       # 48 observation rows per head-instance, window = the last 24 tokens
    (1, 1, 8, 300, 40, 30, 2, F16),        # three row tiles; the window crosses a 128-key tile boundary
    (1, 2, 8, 130, 130, 13, 2, F16),       # the window is the whole context: the first query sees one key
])
@pytest.mark.parametrize("score_kernel", ["tcgen05", "mma_sync"])
def test_observation_window_inside_the_context(B, H, Hq, N, W, R, b, dtype, score_kernel):
    """The observation queries are the last W context tokens, causally masked (each sees the keys up to
    itself): both scoring kernels against the oracle's masked softmax, then the rest of the path."""
    which = kvr.KVR_SCORE_TCGEN05 if score_kernel == "tcgen05" else kvr.KVR_SCORE_MMA_SYNC
    K, V, Q, q = make_case(700 + N, B, H, Hq, N, W, dtype, 1)
    run_and_check(K, V, Q, q, R=R, n_recent=0, b=b, seeds=synth.hash_seeds(N + 2), score_kernel=which,
                  obs_causal=True)


@pytest.mark.parametrize("B,H,Hq,N,W,R,b,dtype,which", [
    (1, 2, 8, 3000, 8, 300, 37, F16, "staged"),      # G = 4, one class
    (1, 2, 8, 6000, 8, 1500, 200, BF16, "staged"),   # 4 x 4 classes, bf16
    (1, 2, 4, 1500, 4, 150, 30, F16, "staged"),      # G = 2
    (1, 2, 8, 2000, 8, 200, 21, F16, "split"),
    (1, 1, 8, 700, 4, 70, 9, BF16, "split"),         # G = 8: the split kernel only
])
def test_mean_combine(B, H, Hq, N, W, R, b, dtype, which):
    """The mean combine of the three cells (an option; the paper takes the median) through both decode
    kernels and the stand-alone reconstruction, against the oracle run with the same option."""
    K, V, Q, q = make_case(1200 + N, B, H, Hq, N, W, dtype, 1)
    run_and_check(K, V, Q, q, R=R, n_recent=0, b=b, seeds=synth.hash_seeds(N + 5), combine="mean",
                  decode_kernel=kvr.KVR_DECODE_STAGED if which == "staged" else kvr.KVR_DECODE_SPLIT)


def test_scoring_kernels_agree():
    """Same inputs through both scoring kernels: the scores differ only by fp32 summation order."""
    K, V, Q, q = make_case(55, 2, 4, 16, 3001, 32, F16, 1)
    sk = kvr.kvr_sketch_create(b=20, batch=2, n_layers=1, n_kv_heads=4, n_q_heads=16, max_context=3001,
                               kv_dtype=F16, hash_seeds=synth.hash_seeds(9))
    got = {}
    for which in (kvr.KVR_SCORE_TCGEN05, kvr.KVR_SCORE_MMA_SYNC):
        kvr.kvr_sketch_set_score_kernel(sk, which)
        kvr.kvr_compress(sk, 0, K[0].cuda(), V[0].cuda(), Q[0].cuda(), 300, 0)
        assert kvr.kvr_last_score_kernel(sk) == which
        got[which] = kvr.kvr_get_scores(sk, 0).cpu().numpy()
    assert kvr.kvr_sketch_device_status(sk) == 0
    np.testing.assert_allclose(got[kvr.KVR_SCORE_TCGEN05], got[kvr.KVR_SCORE_MMA_SYNC], rtol=2e-5, atol=1e-9)
    kvr.kvr_sketch_destroy(sk)


def test_staged_kernel_skewed_classes():
    """Raw-index hashing with the same multiplier in every row puts each token's three cells at the
    same index, so only the diagonal classes are populated and each is several times larger than the
    library plans for: the staged kernel has to walk such a class in several chunks."""
    N = 6000
    K, V, Q, q = make_case(4242, 1, 2, 8, N, 8, F16, 1)
    run_and_check(K, V, Q, q, R=600, n_recent=0, b=200, seeds=synth.injective_seeds(), index_mix=False,
                  decode_kernel=kvr.KVR_DECODE_STAGED)


def test_staged_kernel_shared_memory_full():
    """A sketch that nearly fills shared memory by itself (b = 68 in one class) with long class lists:
    the token entries no longer fit at once and the launch must still respect the 227 KB limit."""
    B, H, Hq, N, R, b = 8, 8, 32, 8192, 2048, 68
    K, V, Q, q = make_case(777, B, H, Hq, N, 8, F16, 1)
    run_and_check(K, V, Q, q, R=R, n_recent=0, b=b, seeds=synth.hash_seeds(68), sample_inst=[0, 37, 63],
                  decode_kernel=kvr.KVR_DECODE_STAGED, check_reconstruct=False)


def test_staged_and_split_kernels_agree():
    """Same handle, same inputs, both decode kernels: they differ only in summation order."""
    seeds = synth.hash_seeds(123)
    K, V, Q, q = make_case(77, 1, 4, 16, 5000, 8, F16, 1)
    sk = kvr.kvr_sketch_create(b=50, batch=1, n_layers=1, n_kv_heads=4, n_q_heads=16, max_context=5000,
                               kv_dtype=F16, hash_seeds=seeds)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].cuda(), V[0].cuda(), Q[0].cuda(), 500, 20)
    outs = {}
    for which in (kvr.KVR_DECODE_SPLIT, kvr.KVR_DECODE_STAGED, kvr.KVR_DECODE_SPLIT, kvr.KVR_DECODE_STAGED):
        kvr.kvr_sketch_set_decode_kernel(sk, which)
        out = kvr.kvr_decode_attention(sk, 0, q[0].cuda(), Kr, Vr, ret)
        assert kvr.kvr_last_decode_kernel(sk) == which
        if which in outs:
            assert torch.equal(outs[which], out), "a decode kernel is not reproducible"
        outs[which] = out
    assert (outs[kvr.KVR_DECODE_SPLIT] - outs[kvr.KVR_DECODE_STAGED]).abs().max().item() <= 1e-4
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("N,R,n_recent,b,W", [
    (64, 64, 0, 3, 4),      # 100 % budget: nothing compressed
    (65, 200, 5, 3, 4),     # budget above N
    (96, 0, 0, 5, 4),       # nothing retained: every token reconstructed
    (80, 11, 11, 4, 1),     # whole budget to Recent, a single observation query
    (1, 1, 0, 1, 1),        # one token
    (1, 0, 0, 1, 1),        # one token, compressed
    (50, 5, 0, 1, 2),       # one cell per row: all compressed tokens collide
    (129, 13, 0, 8192, 2),  # the widest sketch
])
def test_edge_cases(N, R, n_recent, b, W):
    K, V, Q, q = make_case(500 + N + R, 1, 2, 8, N, W, F16, 1)
    run_and_check(K, V, Q, q, R=R, n_recent=n_recent, b=b, seeds=synth.hash_seeds(N + 1))


def _sdpa64(q, K, V, H):
    """Textbook attention in fp64 on the CPU (library routine), GQA by repeating kv heads."""
    G = q.shape[-2] // H
    Kf = K.double().repeat_interleave(G, dim=-3)
    Vf = V.double().repeat_interleave(G, dim=-3)
    return torch.nn.functional.scaled_dot_product_attention(q.double().unsqueeze(-2), Kf, Vf).squeeze(-2)


def test_full_budget_equals_textbook_attention():
    K, V, Q, q = make_case(7, 2, 2, 8, 300, 8, F16, 1)
    out_g, _ = run_and_check(K, V, Q, q, R=300, n_recent=0, b=6, seeds=synth.hash_seeds(3))
    want = _sdpa64(q[0], K[0], V[0], 2).reshape(-1, 4, 128).numpy()
    assert np.abs(out_g - want).max() <= TOL


def test_injective_sketch_equals_textbook_attention():
    """Collision-free hashing (raw indices, A=1, C=0, b >= N): reconstruction is exact, so decode over
    10 % retained + 90 % reconstructed tokens equals full attention."""
    N = 400
    K, V, Q, q = make_case(8, 1, 2, 8, N, 8, BF16, 1)
    out_g, _ = run_and_check(K, V, Q, q, R=40, n_recent=4, b=512, seeds=synth.injective_seeds(),
                             index_mix=False)
    want = _sdpa64(q[0], K[0], V[0], 2).reshape(-1, 4, 128).numpy()
    assert np.abs(out_g - want).max() <= TOL


@pytest.mark.parametrize("which", ["split", "staged"])
def test_tokens_appended_after_compress(which):
    """Decode after generation has gone on: tokens newer than the compressed context are kept exactly
    (Recent part) and appended to the retained rows; the softmax covers context and new tokens."""
    B, H, Hq, N, R, b, n_new = 1, 2, 8, 1200, 120, 9, 37
    seeds = synth.hash_seeds(55)
    K, V, Q, q = make_case(606, B, H, Hq, N + n_new, 8, F16, 1)
    Kc, Vc = K[0, :, :, :N].contiguous(), V[0, :, :, :N].contiguous()
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N,
                               kv_dtype=F16, hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, Kc.cuda(), Vc.cuda(), Q[0].cuda(), R, 10)
    Kr2 = torch.cat([Kr, K[0, :, :, N:].cuda()], dim=2).contiguous()
    Vr2 = torch.cat([Vr, V[0, :, :, N:].cuda()], dim=2).contiguous()
    new_idx = torch.arange(N, N + n_new, dtype=torch.int32, device="cuda").expand(B, H, n_new)
    ret2 = torch.cat([ret, new_idx], dim=2).contiguous()
    out = kvr.kvr_decode_attention(sk, 0, q[0].cuda(), Kr2, Vr2, ret2)
    cmp_idx = kvr.kvr_get_assignment(sk, 0)[0].reshape(B * H, -1).cpu().numpy()
    cells_o = orc.insert(inst_major(Kc), inst_major(Vc), cmp_idx, seeds, b)
    want = orc.decode(dec_to_inst(q[0], H), inst_major(Kr2), inst_major(Vr2), ret2.reshape(B * H, -1).cpu().numpy(),
                      cells_o, N + n_new, seeds)
    assert np.abs(out.reshape(B * H, Hq // H, 128).cpu().numpy() - want).max() <= TOL
    with pytest.raises(kvr.KvrError):              # fewer rows than the compress retained
        kvr.kvr_decode_attention(sk, 0, q[0].cuda(), Kr[:, :, :R - 1].contiguous(), Vr[:, :, :R - 1].contiguous(), ret)
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("which,dtype", [("split", F16), ("staged", F16), ("staged", BF16)])
def test_generation_after_compress_scores_and_overflow(which, dtype):
    """Compress, then two rounds of: append exact tokens, decode, accumulate the attention mass of the
    stored rows, overflow step (losers go to the sketch).  Every stage against the oracle: the mass, the
    rows that stay (bit-exact given the scores the kernel produced), the cells, the token lists, and
    the next decode."""
    B, H, Hq, N, R, b, n_rec = 1, 2, 8, 1500, 150, 11, 20
    G = Hq // H
    seeds = synth.hash_seeds(808)
    per_round = (23, 40)
    K, V, Q, q = make_case(909, B, H, Hq, N + sum(per_round), 8, dtype, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N + sum(per_round),
                               kv_dtype=dtype, hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
    Kall, Vall = inst_major(K[0]), inst_major(V[0])                           # [n_inst, N_total, D] float32
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0, :, :, :N].contiguous().to(dev), V[0, :, :, :N].contiguous().to(dev),
                                   Q[0].to(dev), R, n_rec)
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(B * H, -1).cpu().numpy()
    cells_o = orc.insert(Kall[:, :N], Vall[:, :N], cmp0, seeds, b)
    acc = torch.zeros((B, H, R), dtype=torch.float32, device=dev)
    ctx = N
    for rnd, n_new in enumerate(per_round):
        Kr = torch.cat([Kr, K[0, :, :, ctx:ctx + n_new].to(dev)], dim=2).contiguous()
        Vr = torch.cat([Vr, V[0, :, :, ctx:ctx + n_new].to(dev)], dim=2).contiguous()
        new_idx = torch.arange(ctx, ctx + n_new, dtype=torch.int32, device=dev).expand(B, H, n_new)
        ret = torch.cat([ret, new_idx], dim=2).contiguous()
        acc = torch.cat([acc, torch.zeros((B, H, n_new), dtype=torch.float32, device=dev)], dim=2).contiguous()
        ctx += n_new
        qd = synth.make_decode_q(1000 + rnd, B, Hq, 128, dtype, dev)
        out = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
        before = acc.clone()
        kvr.kvr_accumulate_scores(sk, 0, qd, Kr, acc)
        # ---- oracle: decode and mass over the same storage
        ret_np = ret.reshape(B * H, -1).cpu().numpy()
        qo = dec_to_inst(qd, H)
        want = orc.decode(qo, inst_major(Kr), inst_major(Vr), ret_np, cells_o, ctx, seeds)
        assert np.abs(out.reshape(B * H, G, 128).cpu().numpy() - want).max() <= TOL
        mass = orc.decode_mass(qo, inst_major(Kr), inst_major(Vr), ret_np, cells_o, ctx, seeds)
        mass_rows = np.take_along_axis(mass, ret_np.astype(np.int64), axis=1)
        got = (acc - before).reshape(B * H, -1).cpu().numpy()
        np.testing.assert_allclose(got, mass_rows, rtol=2e-3, atol=2e-6)
        # ---- overflow step, decided on the scores the kernel accumulated
        acc_np = acc.reshape(B * H, -1).cpu().numpy()
        keep_o, evict_o, cells_o = orc.demote(inst_major(Kr), inst_major(Vr), ret_np, acc_np, cells_o, R, n_rec, seeds)
        Kr2, Vr2, ret2, acc2 = kvr.kvr_demote(sk, 0, Kr, Vr, ret, acc, ctx, R, n_rec)
        assert (ret2.reshape(B * H, -1).cpu().numpy() == np.take_along_axis(ret_np, keep_o.astype(np.int64), axis=1)).all()
        assert (inst_major(Kr2) == np.take_along_axis(inst_major(Kr), keep_o[:, :, None].astype(np.int64), axis=1)).all()
        assert (inst_major(Vr2) == np.take_along_axis(inst_major(Vr), keep_o[:, :, None].astype(np.int64), axis=1)).all()
        assert (acc2.reshape(B * H, -1).cpu().numpy() == np.take_along_axis(acc_np, keep_o.astype(np.int64), axis=1)).all()
        cells_g = kvr.kvr_get_cells(sk, 0).reshape(B * H, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4)
        assert np.abs(cells_g - cells_o).max() <= TOL
        cmp_g = kvr.kvr_get_assignment(sk, 0)[0].reshape(B * H, -1).cpu().numpy()
        for u in range(B * H):
            want_cmp = np.setdiff1d(np.arange(ctx), ret2.reshape(B * H, -1)[u].cpu().numpy())
            assert (cmp_g[u] == want_cmp).all()
        Kr, Vr, ret, acc = Kr2, Vr2, ret2, acc2
        out2 = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)               # the lists were rebuilt: decode again
        want2 = orc.decode(qo, inst_major(Kr), inst_major(Vr), ret.reshape(B * H, -1).cpu().numpy(), cells_o, ctx, seeds)
        assert np.abs(out2.reshape(B * H, G, 128).cpu().numpy() - want2).max() <= TOL
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("which,dtype,H,Hq,N,b,skew", [("staged", F16, 2, 8, 1800, 40, False), ("staged", BF16, 2, 4, 1800, 9, False),
                                                       ("staged", F16, 2, 2, 6000, 200, True), ("split", F16, 2, 8, 1800, 40, False),
                                                       ("split", BF16, 1, 8, 1800, 12, False)])
def test_scored_decode_keeps_the_scores_of_the_step(which, dtype, H, Hq, N, b, skew):
    """The decode call that also accumulates the step's attention mass (Calculation Phase: the scores of
    the step are kept, not computed again): output, row scores and vague-token scores against the oracle,
    and against the three separate calls on a second handle in the same state.  Two layers in one call
    (head-instances of the call and of the handle are numbered differently), appended rows, and a hashing
    that overfills single classes so that the staged kernel takes its tokens in several stretches."""
    L, B, R, n_new = 2, 1, N // 10, 13
    G = Hq // H
    seeds = synth.injective_seeds() if skew else synth.hash_seeds(4242)
    K, V, Q, q = make_case(4243, B, H, Hq, N + n_new, 8, dtype, L)
    dev = "cuda"
    n_inst = L * B * H
    state = []
    for _ in range(2):
        sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N + n_new,
                                   kv_dtype=dtype, hash_seeds=seeds, index_mix=not skew)
        kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
        Kr, Vr, ret = kvr.kvr_compress(sk, kvr.KVR_ALL_LAYERS, K[..., :N, :].contiguous().to(dev),
                                       V[..., :N, :].contiguous().to(dev), Q.to(dev), R, 10)
        state.append((sk, Kr, Vr, ret))
    sk, Kr, Vr, ret = state[0]
    cmp0 = kvr.kvr_get_assignment(sk, kvr.KVR_ALL_LAYERS)[0].reshape(n_inst, -1).cpu().numpy()
    cells_o = orc.insert(inst_major(K)[:, :N], inst_major(V)[:, :N], cmp0, seeds, b, mix=not skew)
    Kr = torch.cat([Kr, K[..., N:, :].to(dev)], dim=3).contiguous()
    Vr = torch.cat([Vr, V[..., N:, :].to(dev)], dim=3).contiguous()
    ret = torch.cat([ret, torch.arange(N, N + n_new, dtype=torch.int32, device=dev).expand(L, B, H, n_new)], dim=3).contiguous()
    ret_np = ret.reshape(n_inst, -1).cpu().numpy()
    rows = R + n_new
    outs, accs, toks = [], [], []
    for step in range(2):                                   # the second step reuses the workspace of the first
        qd = synth.make_decode_q(4250 + step, L * B, Hq, 128, dtype, dev).reshape(L, B, Hq, 128)
        qo = dec_to_inst(qd, H)
        want = orc.decode(qo, inst_major(Kr), inst_major(Vr), ret_np, cells_o, N + n_new, seeds, mix=not skew)
        mass = orc.decode_mass(qo, inst_major(Kr), inst_major(Vr), ret_np, cells_o, N + n_new, seeds,
                               mix=not skew)
        for k, (h, _, _, _) in enumerate(state):
            acc = torch.full((L, B, H, rows), 0.25, dtype=torch.float32, device=dev)
            s0 = kvr.kvr_get_scores(h, kvr.KVR_ALL_LAYERS).reshape(n_inst, -1).cpu().numpy()
            if k == 0:
                out = kvr.kvr_decode_attention_scored(h, kvr.KVR_ALL_LAYERS, qd, Kr, Vr, ret, acc)
            else:
                out = kvr.kvr_decode_attention(h, kvr.KVR_ALL_LAYERS, qd, Kr, Vr, ret)
                kvr.kvr_accumulate_scores(h, kvr.KVR_ALL_LAYERS, qd, Kr, acc)
                kvr.kvr_accumulate_vague_scores(h, kvr.KVR_ALL_LAYERS, qd)
            assert kvr.kvr_last_decode_kernel(h) == (kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
            assert kvr.kvr_sketch_device_status(h) == 0
            s1 = kvr.kvr_get_scores(h, kvr.KVR_ALL_LAYERS).reshape(n_inst, -1).cpu().numpy()
            assert np.abs(out.reshape(n_inst, G, 128).cpu().numpy() - want).max() <= TOL
            got_rows = acc.reshape(n_inst, rows).cpu().numpy() - 0.25
            np.testing.assert_allclose(got_rows, np.take_along_axis(mass, ret_np.astype(np.int64), axis=1), rtol=2e-3, atol=2e-6)
            for u in range(n_inst):
                np.testing.assert_allclose(s1[u, cmp0[u]] - s0[u, cmp0[u]], mass[u, cmp0[u]], rtol=2e-3, atol=2e-6)
                assert (s1[u, ret_np[u, :R]] == s0[u, ret_np[u, :R]]).all()        # stored tokens: untouched
            outs.append(out.clone()); accs.append(got_rows); toks.append(s1 - s0)
        np.testing.assert_allclose(accs[-2], accs[-1], rtol=2e-4, atol=1e-6)      # one call against the three
        np.testing.assert_allclose(toks[-2], toks[-1], rtol=2e-4, atol=1e-6)
        assert torch.equal(outs[-2], outs[-1])
    for h, _, _, _ in state:
        kvr.kvr_sketch_destroy(h)


@pytest.mark.parametrize("which,dtype,rate", [("staged", F16, 1.1), ("split", BF16, 1.0), ("staged", F16, 0.9)])
def test_swap_loop_and_vague_scores(which, dtype, rate):
    """Algorithm 3's swap loop on the GPU against the oracle: decode, add the attention mass of the
    vague tokens to the per-token scores and of the stored rows to the row scores, then swap.  Which
    tokens change places is an integer decision taken in fp32 on both sides from the scores the kernels
    accumulated, so it is compared exactly; cells within the tolerance; a revived row is the queried
    vector rounded to the cache type (half a unit in the last place of that type, plus the tolerance);
    the next decode is compared with the oracle on the GPU's storage."""
    B, H, Hq, N, R, b, n_rec = 1, 2, 8, 1200, 160, 40, 16
    G = Hq // H
    seeds = synth.hash_seeds(515)
    K, V, Q, q = make_case(616, B, H, Hq, N, 8, dtype, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=dtype,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
    Kall, Vall = inst_major(K[0]), inst_major(V[0])
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].to(dev), V[0].to(dev), Q[0].to(dev), R, n_rec)
    n_inst = B * H
    ret_np = ret.reshape(n_inst, -1).cpu().numpy()
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(n_inst, -1).cpu().numpy()
    cells_o = orc.insert(Kall, Vall, cmp0, seeds, b)
    s0 = kvr.kvr_get_scores(sk, 0).reshape(n_inst, N).clone()
    acc = torch.gather(s0, 1, ret.reshape(n_inst, -1).long()).reshape(B, H, R).contiguous()   # row scores = compress scores
    # ---- one decode step; its mass raises the scores of stored rows and of vague tokens
    qd = synth.make_decode_q(2024, B, Hq, 128, dtype, dev)
    kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
    kvr.kvr_accumulate_scores(sk, 0, qd, Kr, acc)
    kvr.kvr_accumulate_vague_scores(sk, 0, qd)
    qo = dec_to_inst(qd, H)
    mass = orc.decode_mass(qo, inst_major(Kr), inst_major(Vr), ret_np, cells_o, N, seeds)
    s1 = kvr.kvr_get_scores(sk, 0).reshape(n_inst, N).cpu().numpy()
    for u in range(n_inst):
        got = s1[u, cmp0[u]] - s0[u].cpu().numpy()[cmp0[u]]
        np.testing.assert_allclose(got, mass[u, cmp0[u]], rtol=2e-3, atol=2e-6)
        assert (s1[u, ret_np[u]] == s0[u].cpu().numpy()[ret_np[u]]).all()      # stored tokens: untouched here
    # ---- the swap loop
    acc_np = acc.reshape(n_inst, -1).cpu().numpy().copy()
    Kr_b, Vr_b = inst_major(Kr).copy(), inst_major(Vr).copy()
    rounder = lambda x: torch.from_numpy(np.asarray(x, np.float64)).to(dtype).double().numpy()
    limit = 25
    n_sw = kvr.kvr_swap(sk, 0, Kr, Vr, ret, acc, n_rec, rate, limit).reshape(n_inst).cpu().numpy()
    assert kvr.kvr_sketch_device_status(sk) == 0
    ret_g, acc_g = ret.reshape(n_inst, -1).cpu().numpy(), acc.reshape(n_inst, -1).cpu().numpy()
    s2 = kvr.kvr_get_scores(sk, 0).reshape(n_inst, N).cpu().numpy()
    cells_g = kvr.kvr_get_cells(sk, 0).reshape(n_inst, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4)
    cmp_g = kvr.kvr_get_assignment(sk, 0)[0].reshape(n_inst, -1).cpu().numpy()
    ulp = 2.0 ** -11 if dtype == F16 else 2.0 ** -8                            # half a unit in the last place, relative
    new_cells = []
    for u in range(n_inst):
        Ko, Vo, ro, so, to, co, n = orc.swap(Kr_b[u], Vr_b[u], ret_np[u], acc_np[u], s1[u], cells_o[u], n_rec, rate,
                                             limit, seeds, round_rows=rounder)
        assert n == n_sw[u] and n > 0
        assert (ret_g[u] == ro).all() and (acc_g[u] == so).all()
        vague = np.setdiff1d(np.arange(N), ro)
        assert (cmp_g[u] == vague).all()
        assert (s2[u, vague] == to[vague]).all()
        assert np.abs(cells_g[u] - co).max() <= TOL
        dk, dv = np.abs(inst_major(Kr)[u] - Ko), np.abs(inst_major(Vr)[u] - Vo)
        assert (dk <= TOL + 2 * ulp * np.abs(Ko)).all() and (dv <= TOL + 2 * ulp * np.abs(Vo)).all()
        if rate >= 1.0:                      # (below one a token can leave and come back: its row is then a queried one)
            untouched = ro == ret_np[u]
            assert (inst_major(Kr)[u][untouched] == Kr_b[u][untouched]).all()
        new_cells.append(co)
    # ---- the lists were rebuilt: the next decode sees the swapped storage
    out = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
    want = orc.decode(qo, inst_major(Kr), inst_major(Vr), ret_g, np.stack(new_cells), N, seeds)
    assert np.abs(out.reshape(n_inst, G, 128).cpu().numpy() - want).max() <= TOL
    kvr.kvr_sketch_destroy(sk)


def test_swap_loop_with_equal_candidate_scores():
    """Thousands of candidates with the same score: which of them the swap loop gives up is decided by
    the token index alone (the lowest first), and the selection cannot keep all the ties in its
    scratch.  Row indices, row scores and the number of swaps against the oracle, exactly."""
    B, H, Hq, N, R, b, n_rec, limit = 1, 2, 2, 6000, 3200, 60, 8, 40
    seeds = synth.hash_seeds(717)
    K, V, Q, q = make_case(718, B, H, Hq, N, 8, F16, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=F16,
                               hash_seeds=seeds)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].to(dev), V[0].to(dev), Q[0].to(dev), R, n_rec)
    n_inst = B * H
    ret_np = ret.reshape(n_inst, -1).cpu().numpy().copy()
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(n_inst, -1).cpu().numpy()
    cells_o = orc.insert(inst_major(K[0]), inst_major(V[0]), cmp0, seeds, b)
    s1 = kvr.kvr_get_scores(sk, 0).reshape(n_inst, N).cpu().numpy()
    acc = torch.full((B, H, R), 1e-12, dtype=torch.float32, device=dev)          # every candidate the same, below every vague token
    acc_np = acc.reshape(n_inst, -1).cpu().numpy().copy()
    Kr_b, Vr_b = inst_major(Kr).copy(), inst_major(Vr).copy()
    rounder = lambda x: torch.from_numpy(np.asarray(x, np.float64)).to(F16).double().numpy()
    n_sw = kvr.kvr_swap(sk, 0, Kr, Vr, ret, acc, n_rec, 1.1, limit).reshape(n_inst).cpu().numpy()
    assert kvr.kvr_sketch_device_status(sk) == 0
    for u in range(n_inst):
        Ko, Vo, ro, so, to, co, n = orc.swap(Kr_b[u], Vr_b[u], ret_np[u], acc_np[u], s1[u], cells_o[u], n_rec, 1.1, limit,
                                             seeds, round_rows=rounder)
        assert n == n_sw[u] == limit
        assert (ret.reshape(n_inst, -1)[u].cpu().numpy() == ro).all()
        assert (acc.reshape(n_inst, -1)[u].cpu().numpy() == so).all()
        assert (ro[:limit] != ret_np[u][:limit]).all()                           # the lowest token indices went
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("which,dtype,one_call", [("staged", F16, False), ("split", BF16, False), ("staged", BF16, True),
                                                  ("split", F16, True)])
def test_append_runs_algorithm_3_over_several_slack_periods(which, dtype, one_call):
    """kvr_append against the oracle's compress_stream: a generation loop of decode, score
    accumulation (stored rows and vague tokens; as three calls, or kept by the decode call itself) and
    one kvr_append per step, through more than three Slack periods.  Which rows stay and which tokens
    are swapped are integer decisions taken in fp32 from the scores the kernels accumulated, so row
    indices, row scores and per-token scores are compared exactly; cells and rows within the tolerance;
    the decode of every step is compared with the oracle on the storage of that step."""
    drops, swaps = run_stream_case(which=which, dtype=dtype, one_call=one_call, B=1, H=2, Hq=8, N=1000, R=120, b=30, n_rec0=10,
                                   r_budget=10, c_budget=110, slack=6, steps=[3, 1, 2, 4, 1, 3, 2, 2, 4, 1, 3, 2], rate=1.1,
                                   max_swaps=20, seed=4711)
    assert drops >= 3 and swaps > 0


@pytest.mark.parametrize("Qn,dtype,causal,b,N0,R", [
    (1, F16, True, 20, 1200, 150),          # one query: the single-query result
    (4, F16, True, 20, 1200, 150),          # 16 query rows: every warp on its own
    (4, BF16, False, 20, 1200, 150),
    (16, F16, True, 200, 5000, 900),        # 64 query rows: teams of four warps share a tile; 4 x 4 classes
    (8, BF16, True, 64, 3000, 400),         # 32 query rows: teams of two
    (17, F16, False, 33, 2000, 300),        # 68 query rows: a launch of 64 and one of 16 (4 rows used)
    (16, BF16, True, 20, 700, 100),
    (3, F16, True, 37, 900, 0),             # nothing retained but the queries' own tokens; 12 rows (padded to 16)
])
def test_multi_query_decode_against_the_oracle(Qn, dtype, causal, b, N0, R):
    """kvr_decode_attention_mq: Qn queries per head over the compressed cache plus the queries' own
    tokens as appended exact rows, against the oracle's decode_mq (cache rebuilt, every query with its
    own mask), within the tolerance; Qn = 1 also against the single-query entry point."""
    B, H, Hq = 1, 2, 8
    G = Hq // H
    n_inst = B * H
    seeds = synth.hash_seeds(3300 + Qn)
    K, V, Q, _ = make_case(3301 + Qn, B, H, Hq, N0 + Qn, 8, dtype, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N0 + Qn, kv_dtype=dtype,
                               hash_seeds=seeds)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0, :, :, :N0].contiguous().to(dev), V[0, :, :, :N0].contiguous().to(dev),
                                   Q[0].to(dev), R, 0)
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(n_inst, -1).cpu().numpy()
    cells_o = orc.insert(inst_major(K[0])[:, :N0], inst_major(V[0])[:, :N0], cmp0, seeds, b)
    Kr2 = torch.cat([Kr, K[0, :, :, N0:].to(dev)], dim=2).contiguous()
    Vr2 = torch.cat([Vr, V[0, :, :, N0:].to(dev)], dim=2).contiguous()
    ret2 = torch.cat([ret, torch.arange(N0, N0 + Qn, dtype=torch.int32, device=dev).expand(B, H, Qn)], dim=2).contiguous()
    gen = torch.Generator().manual_seed(3302 + Qn)
    qm = torch.randn((B, Hq, Qn, 128), generator=gen).to(dtype)
    out = kvr.kvr_decode_attention_mq(sk, 0, qm.to(dev), Kr2, Vr2, ret2, causal=causal)
    torch.cuda.synchronize()
    assert kvr.kvr_sketch_device_status(sk) == 0
    q_inst = qm.float().reshape(B, H, G, Qn, 128).reshape(n_inst, G, Qn, 128).numpy()
    want = orc.decode_mq(q_inst, inst_major(Kr2), inst_major(Vr2), ret2.reshape(n_inst, -1).cpu().numpy(), cells_o,
                         N0 + Qn, seeds, causal=causal)
    got = out.reshape(B, H, G, Qn, 128).reshape(n_inst, G, Qn, 128).cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= TOL, np.abs(got - want).max()
    if Qn == 1:
        single = kvr.kvr_decode_attention(sk, 0, qm[:, :, 0].contiguous().to(dev), Kr2, Vr2, ret2)
        assert (single - out[:, :, 0]).abs().max().item() <= TOL
    again = kvr.kvr_decode_attention_mq(sk, 0, qm.to(dev), Kr2, Vr2, ret2, causal=causal)      # bit-reproducible
    assert torch.equal(out, again)
    kvr.kvr_sketch_destroy(sk)


def test_multi_query_decode_needs_a_class_grid():
    """A handle with 8 query heads per kv head has no class grid: the multi-query call says so."""
    seeds = synth.hash_seeds(3400)
    K, V, Q, _ = make_case(3401, 1, 1, 8, 300, 4, F16, 1)
    sk = kvr.kvr_sketch_create(b=5, batch=1, n_layers=1, n_kv_heads=1, n_q_heads=8, max_context=300, kv_dtype=F16,
                               hash_seeds=seeds)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].cuda(), V[0].cuda(), Q[0].cuda(), 30, 0)
    qm = torch.randn((1, 8, 2, 128)).to(F16).cuda()
    with pytest.raises(kvr.KvrError) as e:
        kvr.kvr_decode_attention_mq(sk, 0, qm, Kr, Vr, ret, causal=False)
    assert e.value.status == 2
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("which", ["staged", "split"])
def test_hash_seeds_per_kv_head(which):
    """One set of hash seeds per kv head (the head-instances of a kv head share it across batch and
    layers): bucket and sign assignment, cells, reconstruction, decode, the attention mass of vague
    tokens, an overflow step and several queries per head, each head-instance against the oracle run
    with its own head's seeds; the heads really hash differently."""
    B, H, Hq, L, N, W, R, b = 2, 2, 8, 2, 1100, 8, 120, 13
    G = Hq // H
    n_inst = L * B * H
    seeds = np.stack([synth.hash_seeds(7100), synth.hash_seeds(7200)])           # [H, r, 4]
    K, V, Q, q = make_case(7001, B, H, Hq, N + 6, W, F16, L)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N + 6, kv_dtype=F16,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_SPLIT if which == "split" else kvr.KVR_DECODE_STAGED)
    Kd, Vd = K[:, :, :, :N].contiguous().to(dev), V[:, :, :, :N].contiguous().to(dev)
    Kr, Vr, ret = kvr.kvr_compress(sk, kvr.KVR_ALL_LAYERS, Kd, Vd, Q.to(dev), R, 5)
    out = kvr.kvr_decode_attention(sk, kvr.KVR_ALL_LAYERS, q.to(dev), Kr, Vr, ret)
    cmp_g, bk_g, sg_g = (x.cpu().numpy() for x in kvr.kvr_get_assignment(sk, kvr.KVR_ALL_LAYERS))
    cells_g = kvr.kvr_get_cells(sk, kvr.KVR_ALL_LAYERS).reshape(n_inst, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4)
    Kt_g, Vt_g = (x.reshape(n_inst, N - R, 128).cpu().numpy() for x in kvr.kvr_reconstruct(sk, kvr.KVR_ALL_LAYERS))
    assert kvr.kvr_sketch_device_status(sk) == 0
    Kc, Vc = inst_major(K)[:, :N], inst_major(V)[:, :N]
    qc = dec_to_inst(q, H)
    cmp_g, bk_g, sg_g = cmp_g.reshape(n_inst, -1), bk_g.reshape(n_inst, 3, -1), sg_g.reshape(n_inst, 3, -1)
    ret_np, out_np = ret.reshape(n_inst, R).cpu().numpy(), out.reshape(n_inst, G, 128).cpu().numpy()
    Kr_np, Vr_np = inst_major(Kr), inst_major(Vr)
    cells_o = []
    for u in range(n_inst):
        sd = seeds[u % H]
        bo, so = orc.bucket_sign(cmp_g[u], sd, b)
        assert (bk_g[u] == bo).all() and (sg_g[u] == so).all()
        co = orc.insert(Kc[u:u + 1], Vc[u:u + 1], cmp_g[u:u + 1], sd, b)
        cells_o.append(co[0])
        assert np.abs(cells_g[u] - co[0]).max() <= TOL
        Kt_o, Vt_o = orc.query(co, cmp_g[u:u + 1], sd)
        assert np.abs(Kt_g[u] - Kt_o[0]).max() <= TOL and np.abs(Vt_g[u] - Vt_o[0]).max() <= TOL
        want = orc.decode(qc[u:u + 1], Kr_np[u:u + 1], Vr_np[u:u + 1], ret_np[u:u + 1], co, N, sd)
        assert np.abs(out_np[u] - want[0]).max() <= TOL
    u0, u1 = 0, 1                                                               # same batch element and layer, heads 0 and 1
    both = np.intersect1d(cmp_g[u0], cmp_g[u1])
    i0, i1 = np.searchsorted(cmp_g[u0], both), np.searchsorted(cmp_g[u1], both)
    assert (bk_g[u0][:, i0] != bk_g[u1][:, i1]).mean() > 0.5                   # different hash functions per head
    # ---- several queries per head (layer 1) and the streaming side (layer 0) use the same tables
    if which == "staged":
        gen = torch.Generator().manual_seed(7002)
        qm = torch.randn((B, Hq, 3, 128), generator=gen).to(F16)
        om = kvr.kvr_decode_attention_mq(sk, 1, qm.to(dev), Kr[1], Vr[1], ret[1], causal=False)
        qmi = qm.float().reshape(B, H, G, 3, 128).reshape(B * H, G, 3, 128).numpy()
        for k in range(B * H):
            u = B * H + k
            want = orc.decode_mq(qmi[k:k + 1], Kr_np[u:u + 1], Vr_np[u:u + 1], ret_np[u:u + 1], cells_o[u][None], N, seeds[u % H],
                                 causal=False)
            assert np.abs(om.reshape(B * H, G, 3, 128).cpu().numpy()[k] - want[0]).max() <= TOL
    s0 = kvr.kvr_get_scores(sk, 0).reshape(B * H, -1)
    acc = torch.gather(s0, 1, ret[0].reshape(B * H, -1).long()).reshape(B, H, R).contiguous()
    Kn, Vn = K[0, :, :, N:N + 6].contiguous().to(dev), V[0, :, :, N:N + 6].contiguous().to(dev)
    acc_np = acc.reshape(B * H, -1).cpu().numpy()
    tok_np = s0.cpu().numpy()
    Ko, Vo, ro, so, rec, n_sw = kvr.kvr_append(sk, 0, Kr[0], Vr[0], ret[0], acc, 5, Kn, Vn, 4, R - 10, 2, 1.1, 8)
    cells_a = kvr.kvr_get_cells(sk, 0).reshape(B * H, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4)
    for u in range(B * H):
        tok_u = np.concatenate([tok_np[u], np.zeros(6, np.float32)])
        got = orc.compress_stream(Kr_np[u], Vr_np[u], ret_np[u], acc_np[u], 5, tok_u, cells_o[u], inst_major(K[0])[u, N:N + 6],
                                  inst_major(V[0])[u, N:N + 6], np.arange(N, N + 6, dtype=np.int32), 4, R - 10, 2, 1.1, 8,
                                  seeds[u % H], round_rows=lambda x: torch.from_numpy(np.asarray(x, np.float64)).to(F16).double().numpy())
        assert (ro.reshape(B * H, -1).cpu().numpy()[u] == got[2]).all() and got[4] == rec
        assert np.abs(cells_a[u] - got[6]).max() <= TOL
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("r,dtype,Hq,combine", [(1, F16, 8, "median"), (5, F16, 8, "median"), (5, BF16, 16, "median"),
                                               (5, F16, 4, "mean"), (1, BF16, 2, "median")])
def test_sketches_with_one_and_five_rows(r, dtype, Hq, combine):
    """r = 1 (Algorithm 2 is a direct look-up) and r = 5 (middle of five): hashing, cells,
    reconstruction and decode against the oracle, which is generic in r; 1 to 8 query heads per kv
    head, the mean combine, two layers in one call."""
    B, H, L, N, W, R, b = 1, 2, 2, 1300, 8, 140, 17
    K, V, Q, q = make_case(8100 + r, B, H, Hq, N, W, dtype, L)
    seeds = synth.hash_seeds(8200 + r, r=r)
    run_and_check(K, V, Q, q, R=R, n_recent=7, b=b, seeds=seeds, layer_mode="all", combine=combine)


def test_one_row_sketch_without_collisions_is_the_full_cache():
    """r = 1 with one cell per token (raw indices, h(J) = J): every vague token is looked up exactly,
    so the decode equals attention over the uncompressed cache."""
    B, H, Hq, N, W, R = 1, 2, 8, 500, 4, 50
    K, V, Q, q = make_case(8300, B, H, Hq, N, W, F16, 1)
    seeds = synth.injective_seeds()[:1]
    out_g, out_o = run_and_check(K, V, Q, q, R=R, n_recent=0, b=N, seeds=seeds, index_mix=False)
    G = Hq // H
    Kc, Vc, qc = inst_major(K[0]).astype(np.float64), inst_major(V[0]).astype(np.float64), dec_to_inst(q[0], H).astype(np.float64)
    logits = np.einsum("ugd,ujd->ugj", qc, Kc) / math.sqrt(128)
    p = np.exp(logits - logits.max(-1, keepdims=True))
    full = np.einsum("ugj,ujd->ugd", p / p.sum(-1, keepdims=True), Vc)
    assert np.abs(out_g - full).max() <= TOL


def test_calls_written_for_three_rows_say_so():
    """The streaming side, the multi-query call and the allocation-free call serve r = 3 only."""
    K, V, Q, q = make_case(8400, 1, 2, 8, 300, 4, F16, 1)
    sk = kvr.kvr_sketch_create(b=9, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8, max_context=300, r=5, kv_dtype=F16,
                               hash_seeds=synth.hash_seeds(8401, r=5))
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].cuda(), V[0].cuda(), Q[0].cuda(), 30, 0)
    qd = q[0].cuda()
    kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
    for call in (lambda: kvr.kvr_accumulate_vague_scores(sk, 0, qd),
                 lambda: kvr.kvr_decode_attention_static(sk, 0, qd, Kr, Vr, ret),
                 lambda: kvr.kvr_decode_attention_mq(sk, 0, torch.zeros((1, 8, 2, 128), dtype=F16, device="cuda"), Kr, Vr, ret)):
        with pytest.raises(kvr.KvrError) as e:
            call()
        assert e.value.status == 2
    kvr.kvr_sketch_destroy(sk)


def test_bounded_wait_gives_up_and_reports():
    """The staged kernel's wait on its staging barrier is bounded.  With the test hook the kernel expects
    more bytes than its copies deliver, so the barrier never completes: every class CTA waits the
    (shortened) limit, sets the status bit and carries on; the cells had landed long before, so the
    output still matches an untouched handle.  Nothing faults or hangs; normal operation afterwards."""
    seeds = synth.hash_seeds(9100)
    K, V, Q, q = make_case(9101, 1, 2, 8, 2000, 8, F16, 1)
    dev = "cuda"
    outs = []
    for hook in (False, True):
        sk = kvr.kvr_sketch_create(b=25, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8, max_context=2000, kv_dtype=F16,
                                   hash_seeds=seeds)
        kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_STAGED)
        Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0].to(dev), V[0].to(dev), Q[0].to(dev), 200, 0)
        if hook:
            kvr.kvr_sketch_set_wait_test(sk, 1_000_000, 16)                     # 1 ms, 16 bytes that never arrive
        outs.append(kvr.kvr_decode_attention(sk, 0, q[0].to(dev), Kr, Vr, ret).clone())
        assert kvr.kvr_sketch_device_status(sk) == (1 if hook else 0)
        if hook:
            kvr.kvr_sketch_set_wait_test(sk, 200_000_000, 0)
            again = kvr.kvr_decode_attention(sk, 0, q[0].to(dev), Kr, Vr, ret)
            assert torch.equal(again, outs[0])
        kvr.kvr_sketch_destroy(sk)
    assert torch.equal(outs[0], outs[1])
    with pytest.raises(kvr.KvrError):
        sk = kvr.kvr_sketch_create(b=5, batch=1, n_layers=1, n_kv_heads=1, n_q_heads=1, max_context=64, kv_dtype=F16,
                                   hash_seeds=seeds)
        try:
            kvr.kvr_sketch_set_wait_test(sk, 10, 16)                            # a limit that could cut a copy short
        finally:
            kvr.kvr_sketch_destroy(sk)


def test_bounded_wait_of_the_scoring_kernel_gives_up_and_reports():
    """The tcgen05 scoring kernel's waits are bounded too.  With the hook its wait for the query tile
    runs out: status bit 1, the CTA runs to its end and releases its tensor memory, nothing faults or
    hangs; with the hook off again the same handle compresses normally and matches the oracle."""
    seeds = synth.hash_seeds(9200)
    B, H, Hq, N, W, R, b = 1, 2, 8, 1024, 32, 100, 12
    K, V, Q, q = make_case(9201, B, H, Hq, N, W, F16, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=F16,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_score_kernel(sk, kvr.KVR_SCORE_TCGEN05)
    kvr.kvr_sketch_set_wait_test(sk, 1_000_000, 16)
    kvr.kvr_compress(sk, 0, K[0].to(dev), V[0].to(dev), Q[0].to(dev), R, 0)
    assert kvr.kvr_last_score_kernel(sk) == kvr.KVR_SCORE_TCGEN05
    assert kvr.kvr_sketch_device_status(sk) & 2
    kvr.kvr_sketch_destroy(sk)
    # a fresh handle (the status word is sticky), hook set and taken back: normal operation
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=F16,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_score_kernel(sk, kvr.KVR_SCORE_TCGEN05)
    kvr.kvr_sketch_set_wait_test(sk, 1_000_000, 16)
    kvr.kvr_sketch_set_wait_test(sk, 200_000_000, 0)
    kvr.kvr_compress(sk, 0, K[0].to(dev), V[0].to(dev), Q[0].to(dev), R, 0)
    assert kvr.kvr_sketch_device_status(sk) == 0
    got = kvr.kvr_get_scores(sk, 0).reshape(B * H, N).cpu().numpy()
    want = orc.scores(obs_to_inst(Q[0], H), inst_major(K[0]))
    kvr.kvr_sketch_destroy(sk)
    np.testing.assert_allclose(got, want, rtol=2e-4, atol=1e-7)


@pytest.mark.parametrize("dtype,score_kernel", [(F16, kvr.KVR_SCORE_TCGEN05), (BF16, kvr.KVR_SCORE_MMA_SYNC)])
def test_peaked_scores_with_sink_tokens(dtype, score_kernel):
    """The structured inputs: four sink tokens per head take a large part of every observation query's softmax
    (a quarter to a half of it on 4 of 3000 tokens), and decode
    queries that look at them too.  Every stage against the oracle; the sinks must be retained."""
    L, B, H, Hq, N, W = 1, 2, 2, 8, 3000, 32
    K, V, Q, q = make_case(6100, B, H, Hq, N, W, dtype, L)
    for layer in range(L):
        synth.plant_sinks(K[layer], Q[layer])
    mean = Q[0].float().reshape(B, H, (Hq // H) * W, 128).mean(dim=2)                      # decode queries lean the same way
    q = (q.float() + 3.0 * mean.repeat_interleave(Hq // H, dim=1)[None]).to(dtype)
    out_g, out_o = run_and_check(K, V, Q, q, R=300, n_recent=16, b=20, seeds=synth.hash_seeds(6101), score_kernel=score_kernel)
    sk = kvr.kvr_sketch_create(b=20, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=dtype,
                               hash_seeds=synth.hash_seeds(6101))
    _, _, ret = kvr.kvr_compress(sk, 0, K[0].cuda(), V[0].cuda(), Q[0].cuda(), 300, 16)
    s = kvr.kvr_get_scores(sk, 0).reshape(B * H, N)
    assert (ret.reshape(B * H, -1)[:, :4].cpu() == torch.arange(4)).all()                    # the sinks are kept
    assert (s[:, :4].sum(dim=1) > 0.2 * s.sum(dim=1)).all()                                  # and hold a large part of the mass (4 of 3000 tokens)
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("seed", range(16))
def test_random_valid_shapes(seed):
    """Shapes, budgets, widths, types, kernels and options drawn at random (seeded) from everything the
    library accepts, each through every stage against the oracle: the cases nobody thought of."""
    rng = np.random.default_rng(1000 + seed)
    L, B = int(rng.choice([1, 1, 2])), int(rng.choice([1, 1, 2, 3]))
    H, G = int(rng.choice([1, 2, 3, 4, 8])), int(rng.choice([1, 2, 4, 4, 8]))
    N = int(rng.integers(*[(1, 40), (40, 700), (700, 4000), (4000, 9000)][int(rng.choice([0, 1, 1, 2, 2, 2, 3]))]))
    W = int(rng.choice([1, 3, 8, 32, 40]))
    R = [0, N, N + 5, int(rng.integers(0, N + 1)), int(rng.integers(0, N + 1)), int(rng.integers(0, N + 1))][int(rng.integers(0, 6))]
    Rr = min(R, N)
    n_recent = int(rng.integers(0, Rr + 1)) if rng.integers(0, 2) else min(Rr, int(rng.integers(0, 17)))
    b = int(rng.choice([1, 2, 7, 16, 64, 137, 273, 300])) if rng.integers(0, 2) else int(rng.integers(1, 301))
    dtype = F16 if rng.integers(0, 2) else BF16
    r = int(rng.choice([3, 3, 3, 3, 1, 5]))
    dk = int(rng.choice([kvr.KVR_DECODE_AUTO, kvr.KVR_DECODE_AUTO, kvr.KVR_DECODE_SPLIT, kvr.KVR_DECODE_STAGED]))
    if (r != 3 or G > 4 or R >= N) and dk == kvr.KVR_DECODE_STAGED:
        dk = kvr.KVR_DECODE_AUTO                                 # (the staged kernel does not serve these: the call would use the other)
    sck = int(rng.choice([kvr.KVR_SCORE_AUTO, kvr.KVR_SCORE_AUTO, kvr.KVR_SCORE_MMA_SYNC]))
    causal = bool(rng.integers(0, 4) == 0) and W <= N
    combine = "mean" if (rng.integers(0, 5) == 0 and r == 3) else "median"
    mix = bool(rng.integers(0, 6) != 0)
    K, V, Q, q = make_case(3000 + seed, B, H, H * G, N, W, dtype, L)
    seeds = synth.hash_seeds(77 + seed, r) if mix else synth.injective_seeds(r)
    run_and_check(K, V, Q, q, R=R, n_recent=n_recent, b=b, seeds=seeds, index_mix=mix,
                  layer_mode="all" if rng.integers(0, 2) else "per_layer", decode_kernel=dk, score_kernel=sck,
                  obs_causal=causal, combine=combine)


@pytest.mark.parametrize("seed", range(6))
def test_random_generation_loops(seed):
    """The same for the streaming side: random storage sizes, Slack, ReplaceRate (below one too), swap
    limits and step sizes, as three calls or with the decode call that keeps the scores.  (Sketches of
    at least 8 cells per row: a swap deletes a queried vector, which carries the rounding error of the
    cells it was read from, from all three of them, so dozens of swaps on the same two or three cells
    double a last-place difference between fp32 and fp64 cells again and again.  That is the
    conditioning of the method on such a sketch, in any precision, not something a tolerance describes.)"""
    rng = np.random.default_rng(2000 + seed)
    H, G, B = int(rng.choice([1, 2, 3])), int(rng.choice([1, 2, 4, 8])), int(rng.choice([1, 2]))
    N = int(rng.integers(60, 2500))
    r_budget = int(rng.integers(1, 40))
    R = min(N, r_budget + int(rng.integers(1, max(2, N // 3))))
    n_rec0 = min(r_budget, R - 1)
    run_stream_case(which="split" if G == 8 or rng.integers(0, 3) == 0 else "staged", dtype=F16 if rng.integers(0, 2) else BF16,
                    one_call=bool(rng.integers(0, 2)), B=B, H=H, Hq=H * G, N=N, R=R, b=int(rng.integers(8, 120)), n_rec0=n_rec0,
                    r_budget=r_budget, c_budget=R - n_rec0, slack=int(rng.integers(0, 9)),
                    steps=[int(x) for x in rng.integers(1, 6, size=int(rng.integers(3, 10)))],
                    rate=float(rng.choice([1.1, 1.0, 1.5, 0.9])), max_swaps=int(rng.choice([0, 1, 5, 20, 300, 600])),
                    seed=9000 + 7 * seed)


def test_per_layer_budgets_in_one_handle():
    """Budgets that differ from layer to layer (kvr_layer_budgets from per-layer weights): every layer
    of one handle is compressed with its own budget and decoded; selection, cells and outputs against
    the oracle run with that layer's budget."""
    B, H, Hq, L, N, W, b = 1, 2, 8, 3, 900, 8, 9
    G = Hq // H
    budgets = kvr.kvr_layer_budgets([4.0, 1.0, 2.5], N, 0.2)
    assert sum(budgets) == 3 * 180 and budgets == orc.layer_budgets([4.0, 1.0, 2.5], N, 0.2)
    seeds = synth.hash_seeds(31)
    K, V, Q, q = make_case(4321, B, H, Hq, N, W, F16, L)
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N, kv_dtype=F16,
                               hash_seeds=seeds)
    stored = [kvr.kvr_compress(sk, l, K[l].cuda(), V[l].cuda(), Q[l].cuda(), budgets[l], 0) for l in range(L)]
    for l in range(L):
        assert kvr.kvr_layer_shape(sk, l) == (N, budgets[l])
        Kr, Vr, ret = stored[l]
        out = kvr.kvr_decode_attention(sk, l, q[l].cuda(), Kr, Vr, ret)
        s_g = kvr.kvr_get_scores(sk, l).reshape(B * H, N).cpu().numpy()
        ret_g = ret.reshape(B * H, -1).cpu().numpy()
        ret_o, cmp_o = orc.select(s_g, budgets[l], 0)
        assert (ret_g == ret_o).all()
        Kc, Vc = inst_major(K[l]), inst_major(V[l])
        cells_o = orc.insert(Kc, Vc, cmp_o, seeds, b)
        want = orc.decode(dec_to_inst(q[l], H), orc.gather(Kc, ret_g), orc.gather(Vc, ret_g), ret_g, cells_o, N, seeds)
        assert np.abs(out.reshape(B * H, G, 128).cpu().numpy() - want).max() <= TOL
    assert kvr.kvr_sketch_device_status(sk) == 0
    kvr.kvr_sketch_destroy(sk)


def test_chained_decode_launches_see_every_change_of_the_storage():
    """Back-to-back staged decode launches are chained (a launch may start staging its cells while the
    previous one drains).  Whatever changes cells or token lists in between has to break the chain:
    compress again with other data, decode, overflow step, decode, all on one stream without any
    synchronisation, and every output must equal what a fresh handle computes for the same storage."""
    B, H, Hq, N, R, b = 1, 2, 8, 2500, 250, 30
    seeds = synth.hash_seeds(77)
    dev = "cuda"

    def fresh(Kd, Vd, Qd, qd):
        sk2 = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N + 64,
                                    kv_dtype=F16, hash_seeds=seeds)
        kvr.kvr_sketch_set_decode_kernel(sk2, kvr.KVR_DECODE_STAGED)
        Kr2, Vr2, ret2 = kvr.kvr_compress(sk2, 0, Kd, Vd, Qd, R, 0)
        out2 = kvr.kvr_decode_attention(sk2, 0, qd, Kr2, Vr2, ret2).clone()
        kvr.kvr_sketch_destroy(sk2)
        return out2

    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N + 64, kv_dtype=F16,
                               hash_seeds=seeds)
    kvr.kvr_sketch_set_decode_kernel(sk, kvr.KVR_DECODE_STAGED)
    data = [tuple(x[0].to(dev) for x in make_case(3000 + i, B, H, Hq, N, 8, F16, 1)) for i in range(2)]
    outs = []
    for K, V, Q, q in data:                      # no synchronisation anywhere in this loop
        Kr, Vr, ret = kvr.kvr_compress(sk, 0, K, V, Q, R, 0)
        for _ in range(3):                       # chained launches on unchanged storage
            outs.append(kvr.kvr_decode_attention(sk, 0, q, Kr, Vr, ret))
    # overflow step between two chained decodes
    K, V, Q, q = data[1]
    acc = torch.rand((B, H, R), dtype=torch.float32, device=dev)
    Kr2, Vr2, ret2, _ = kvr.kvr_demote(sk, 0, Kr, Vr, ret, acc, N, R - 40, 0)
    after = kvr.kvr_decode_attention(sk, 0, q, Kr2, Vr2, ret2)
    after2 = kvr.kvr_decode_attention(sk, 0, q, Kr2, Vr2, ret2)
    torch.cuda.synchronize()
    assert kvr.kvr_sketch_device_status(sk) == 0
    for i, (K, V, Q, q) in enumerate(data):
        want = fresh(K, V, Q, q)
        for j in range(3):
            assert torch.equal(outs[3 * i + j], want), (i, j)      # same kernel, same storage: bit-identical
    assert torch.equal(after, after2) and not torch.equal(after, outs[-1])
    # the storage after the overflow step, through the oracle
    ret_np = ret2.reshape(B * H, -1).cpu().numpy()
    cells_g = kvr.kvr_get_cells(sk, 0).reshape(B * H, 2, 3, b, 128).cpu().numpy().transpose(0, 2, 3, 1, 4).astype(np.float64)
    want = orc.decode(dec_to_inst(q[None][0], H), inst_major(Kr2), inst_major(Vr2), ret_np, cells_g, N, seeds)
    assert np.abs(after.reshape(B * H, Hq // H, 128).cpu().numpy() - want).max() <= TOL
    kvr.kvr_sketch_destroy(sk)


def test_custom_softmax_scale():
    K, V, Q, q = make_case(9, 1, 2, 8, 150, 4, F16, 1)
    run_and_check(K, V, Q, q, R=15, n_recent=0, b=3, seeds=synth.hash_seeds(4), scale=0.05)


def test_config1_single_layer_2k():
    """First benchmark configuration in full: 8 kv heads / 32 q heads, N = 2048, 10 % budget (205),
    b = 7, fp16 with outlier key channels, 32 observation queries."""
    w = synth.WORKLOADS["2k_single_layer"]
    K, V, Q = synth.layer_inputs(w, 0, "cpu")
    q = synth.decode_queries(w, 0, "cpu")
    assert w.budget == 205 and w.b == 7
    run_and_check(K[None], V[None], Q[None], q, R=w.budget, n_recent=0, b=w.b, seeds=synth.hash_seeds(w.seed + 3))


@pytest.mark.parametrize("mode,L", [("per_layer", 1), ("all", 4)])
def test_32k_full_size_sampled(mode, L):
    """Third benchmark configuration at full per-layer size (N = 32768, R = 8192, b = 273) in the launch
    shapes the benchmark uses (one layer per call; several layers per launch); the oracle checks two
    sampled head-instances."""
    w = synth.WORKLOADS["32k_llama3_8b"]
    dev = "cuda"
    Ks, Vs, Qs = zip(*[synth.layer_inputs(w, layer, dev) for layer in range(L)])
    K, V, Q = torch.stack(Ks), torch.stack(Vs), torch.stack(Qs)
    q = synth.decode_queries(w, 0, dev)[:L]
    n_inst = L * w.n_kv_heads
    run_and_check(K.cpu(), V.cpu(), Q.cpu(), q.cpu(), R=w.budget, n_recent=0, b=w.b,
                  seeds=synth.hash_seeds(w.seed + 3), layer_mode=mode, sample_inst=sampled_instances(n_inst, 2, L),
                  expect_decode_kernel=kvr.KVR_DECODE_STAGED)        # the kernel the benchmark times


@pytest.mark.parametrize("name,ratio,mult,n_sample", [
    ("32k_llama3_8b_batch16", 0.0, 0.0, 3),     # bf16, 128 head-instances per layer launch: 2048 class CTAs, many waves
    ("2k_llama3_8b", 0.0, 0.0, 3),              # short context: one class cut into slices per head-instance
] + [("8k_qwen3_8b_batch8", r, m, 1) for r in (0.05, 0.10, 0.25, 0.50) for m in (0.5, 1.0, 2.0)])   # the whole sweep
def test_other_workloads_one_layer_sampled(name, ratio, mult, n_sample):
    """One layer of the other benchmark workloads at full per-layer size, in the launch shape the
    benchmark uses for them (one layer per call), every point of the budget x width sweep included;
    the oracle checks sampled head-instances.  The library has to pick the staged kernel by itself."""
    import dataclasses
    w = synth.WORKLOADS[name]
    if ratio:
        w = dataclasses.replace(w, budget_ratio=ratio, width_mult=mult)
    K, V, Q = synth.layer_inputs(w, 0, "cuda")
    q = synth.decode_queries(w, 0, "cuda")[:1]
    n_inst = w.batch * w.n_kv_heads
    run_and_check(K[None].cpu(), V[None].cpu(), Q[None].cpu(), q.cpu(), R=w.budget, n_recent=0, b=w.b,
                  seeds=synth.hash_seeds(w.seed + 3), sample_inst=sampled_instances(n_inst, n_sample, int(ratio * 100 + mult * 10)),
                  check_reconstruct=False, expect_decode_kernel=kvr.KVR_DECODE_STAGED)


def test_recompress_with_other_shape_and_determinism():
    """A layer can be compressed again with a shorter context; results are bit-reproducible."""
    seeds = synth.hash_seeds(77)
    K, V, Q, q = make_case(31, 1, 2, 8, 900, 16, F16, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=11, batch=1, n_layers=1, n_kv_heads=2, n_q_heads=8, max_context=900,
                               kv_dtype=F16, hash_seeds=seeds)
    Kd, Vd, Qd, qd = (x[0].to(dev) for x in (K, V, Q, q))
    outs, cells = [], []
    for N in (900, 300, 300):
        Kn, Vn = Kd[:, :, :N].contiguous(), Vd[:, :, :N].contiguous()
        Kr, Vr, ret = kvr.kvr_compress(sk, 0, Kn, Vn, Qd, N // 10, 3)
        out = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
        outs.append(out.cpu().numpy())
        cells.append(kvr.kvr_get_cells(sk, 0).cpu().numpy())
        Kc, Vc = inst_major(Kn), inst_major(Vn)
        cmp_idx = kvr.kvr_get_assignment(sk, 0)[0].reshape(2, -1).cpu().numpy()
        cells_o = orc.insert(Kc, Vc, cmp_idx, seeds, 11)
        want = orc.decode(dec_to_inst(q[0], 2), inst_major(Kr), inst_major(Vr), ret.reshape(2, -1).cpu().numpy(),
                          cells_o, N, seeds)
        assert np.abs(out.reshape(2, 4, 128).cpu().numpy() - want).max() <= TOL
    assert (outs[1] == outs[2]).all() and (cells[1] == cells[2]).all()
    kvr.kvr_sketch_destroy(sk)


def test_host_buffer_calls_match_device_calls():
    seeds = synth.hash_seeds(78)
    K, V, Q, q = make_case(41, 2, 2, 8, 500, 8, BF16, 2)
    dev = "cuda"
    mk = lambda: kvr.kvr_sketch_create(b=6, batch=2, n_layers=2, n_kv_heads=2, n_q_heads=8, max_context=500,
                                       kv_dtype=BF16, hash_seeds=seeds)
    sk_d, sk_h = mk(), mk()
    for layer in range(2):
        Kr, Vr, ret = kvr.kvr_compress(sk_d, layer, K[layer].to(dev), V[layer].to(dev), Q[layer].to(dev), 50, 5)
        want = kvr.kvr_decode_attention(sk_d, layer, q[layer].to(dev), Kr, Vr, ret).cpu()
        kvr.kvr_compress_host(sk_h, layer, K[layer].pin_memory(), V[layer].pin_memory(), Q[layer].pin_memory(), 50, 5)
        got = torch.empty(2, 8, 128, dtype=torch.float32).pin_memory()
        kvr.kvr_decode_attention_host(sk_h, layer, q[layer].pin_memory(), got)
        assert torch.equal(got, want)
    got = torch.empty(2, 2, 8, 128, dtype=torch.float32)
    kvr.kvr_decode_attention_host(sk_h, kvr.KVR_ALL_LAYERS, q.contiguous(), got)
    assert np.isfinite(got.numpy()).all()
    kvr.kvr_sketch_destroy(sk_d)
    kvr.kvr_sketch_destroy(sk_h)


def test_runtime_argument_errors():
    seeds = synth.hash_seeds(79)
    sk = kvr.kvr_sketch_create(b=4, batch=1, n_layers=2, n_kv_heads=2, n_q_heads=8, max_context=128,
                               kv_dtype=F16, hash_seeds=seeds)
    K, V, Q, q = (x[0].cuda() for x in make_case(51, 1, 2, 8, 128, 4, F16, 1))
    with pytest.raises(kvr.KvrError) as e:      # decode before compress
        kvr.kvr_decode_attention(sk, 0, q, K[:, :, :8].contiguous(), V[:, :, :8].contiguous(), None)
    assert e.value.status == 6
    with pytest.raises(kvr.KvrError) as e:      # n_recent > budget
        kvr.kvr_compress(sk, 0, K, V, Q, 10, 11)
    assert e.value.status == 3
    with pytest.raises(kvr.KvrError) as e:      # layer out of range
        kvr.kvr_compress(sk, 5, K, V, Q, 10, 0)
    assert e.value.status == 3
    Kr, Vr, ret = kvr.kvr_compress(sk, 1, K, V, Q, 10, 0)
    with pytest.raises(kvr.KvrError) as e:      # wrong retained count
        kvr.kvr_decode_attention(sk, 1, q, Kr[:, :, :9].contiguous(), Vr[:, :, :9].contiguous(), ret)
    assert e.value.status == 3
    with pytest.raises(kvr.KvrError) as e:      # all layers, but layer 0 was never compressed
        kvr.kvr_get_scores(sk, kvr.KVR_ALL_LAYERS)
    assert e.value.status == 6
    out = kvr.kvr_decode_attention(sk, 1, q, Kr, Vr, ret)      # the handle still works
    assert torch.isfinite(out).all()
    # ---- the calls added for generation and for the scoring options
    acc = torch.zeros((1, 2, 10), dtype=torch.float32, device="cuda")
    with pytest.raises(kvr.KvrError) as e:      # the swap loop wants the storage as the compress left it
        kvr.kvr_swap(sk, 1, Kr[:, :, :9].contiguous(), Vr[:, :, :9].contiguous(), ret[:, :, :9].contiguous(),
                     acc[:, :, :9].contiguous(), 0, 1.1, 4)
    assert e.value.status == 3
    with pytest.raises(kvr.KvrError) as e:      # a replace rate must be positive
        kvr.kvr_swap(sk, 1, Kr, Vr, ret, acc, 0, 0.0, 4)
    assert e.value.status == 1
    with pytest.raises(kvr.KvrError) as e:      # vague scores of a layer that was never compressed
        kvr.kvr_accumulate_vague_scores(sk, 0, q)
    assert e.value.status == 6
    kvr.kvr_sketch_set_score_kernel(sk, kvr.KVR_SCORE_TCGEN05)
    with pytest.raises(kvr.KvrError) as e:      # 2 head-instances x 16 observation rows: less than one TMA box
        kvr.kvr_compress(sk, 0, K, V, Q, 10, 0)
    assert e.value.status == 2
    kvr.kvr_sketch_set_score_kernel(sk, kvr.KVR_SCORE_AUTO)
    kvr.kvr_sketch_set_obs_window_causal(sk, True)
    with pytest.raises(kvr.KvrError) as e:      # an in-context window longer than the context
        kvr.kvr_compress(sk, 0, K[:, :, :3].contiguous(), V[:, :, :3].contiguous(), Q, 2, 0)
    assert e.value.status == 3
    kvr.kvr_sketch_set_obs_window_causal(sk, False)
    with pytest.raises(kvr.KvrError):
        kvr.kvr_sketch_set_score_kernel(sk, 7)
    Kr0, Vr0, ret0 = kvr.kvr_compress(sk, 0, K, V, Q, 10, 0)   # after all the refusals the handle still works
    assert kvr.kvr_last_score_kernel(sk) == kvr.KVR_SCORE_MMA_SYNC
    assert torch.isfinite(kvr.kvr_decode_attention(sk, 0, q, Kr0, Vr0, ret0)).all()
    kvr.kvr_sketch_destroy(sk)
