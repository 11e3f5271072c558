"""The allocation-free decode entry point (kvr_decode_attention_static) against the ordinary one.

Some hosts cannot allocate device memory while they decode: their own pool already owns every free
byte, or they cannot afford the device-wide synchronisation of cudaMalloc / cudaFree inside the
decode loop.  For them the library offers a decode call whose scratch is a fixed array inside the
library image.  This file is collected last, so a run that stops at the first failure has already
exercised everything else; it must also pass alone in a fresh process (the first call on a device
performs the one-time address look-up of the scratch array)."""
import numpy as np
import pytest
import torch

import paper_2512_17917_b200 as kvr
from oracle import kvr_oracle as orc
from paper_2512_17917_b200 import synth

from kvr_testlib import TOL, dec_to_inst, inst_major, make_case

pytestmark = pytest.mark.gpu


def test_static_scratch_decode_matches_ordinary_decode_twice():
    seeds = synth.hash_seeds(91)
    L, B, H, Hq, N, W, R, b = 2, 1, 4, 16, 3000, 8, 300, 12
    K, V, Q, q = make_case(61, B, H, Hq, N, W, torch.float16, L)
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=L, n_kv_heads=H, n_q_heads=Hq, max_context=N,
                               kv_dtype=torch.float16, hash_seeds=seeds)
    dev = "cuda"
    Kr, Vr, ret = kvr.kvr_compress(sk, kvr.KVR_ALL_LAYERS, K.to(dev), V.to(dev), Q.to(dev), R, 10)
    q2 = synth.make_decode_q(62, L * B, Hq, 128, torch.float16, dev).reshape(L, B, Hq, 128)
    cmp_g = kvr.kvr_get_assignment(sk, kvr.KVR_ALL_LAYERS)[0].reshape(L * B * H, -1).cpu().numpy()
    cells_o = orc.insert(inst_major(K), inst_major(V), cmp_g, seeds, b)
    for qq in (q.to(dev), q2):                       # two calls in a row share the same scratch array
        want_all = kvr.kvr_decode_attention(sk, kvr.KVR_ALL_LAYERS, qq, Kr, Vr, ret)
        out = torch.full_like(want_all, float("nan"))
        got_all = kvr.kvr_decode_attention_static(sk, kvr.KVR_ALL_LAYERS, qq, Kr, Vr, ret, out=out)
        got_l1 = kvr.kvr_decode_attention_static(sk, 1, qq[1], Kr[1], Vr[1], ret[1])
        want_l1 = kvr.kvr_decode_attention(sk, 1, qq[1], Kr[1], Vr[1], ret[1])
        torch.cuda.synchronize()
        assert torch.isfinite(got_all).all()
        want_o = orc.decode(dec_to_inst(qq, H), inst_major(Kr), inst_major(Vr), ret.reshape(L * B * H, -1).cpu().numpy(),
                            cells_o, N, seeds)
        assert np.abs(got_all.reshape(L * B * H, Hq // H, 128).cpu().numpy() - want_o).max() <= TOL
        assert (got_all - want_all).abs().max().item() <= TOL
        assert (got_l1 - want_l1).abs().max().item() <= TOL
    kvr.kvr_sketch_destroy(sk)


@pytest.mark.parametrize("dtype,H,Hq", [(torch.float16, 2, 8), (torch.bfloat16, 2, 8), (torch.float16, 1, 8)])
def test_static_scratch_decode_with_appended_rows_against_the_oracle(dtype, H, Hq):
    """A generation loop is where a caller that cannot allocate uses this entry point: rows appended
    after the compress are part of the call.  Two calls in a row (the second with more rows), each
    compared with the CPU oracle and with the ordinary entry point; fp16, bf16 and a handle with 8
    query heads per kv head (which the split kernel serves)."""
    B, N, R, b, n_new = 1, 900, 90, 9, (7, 12)
    G = Hq // H
    seeds = synth.hash_seeds(93)
    K, V, Q, q = make_case(66, B, H, Hq, N + sum(n_new), 4, dtype, 1)
    dev = "cuda"
    sk = kvr.kvr_sketch_create(b=b, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=Hq, max_context=N + sum(n_new),
                               kv_dtype=dtype, hash_seeds=seeds)
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K[0, :, :, :N].contiguous().to(dev), V[0, :, :, :N].contiguous().to(dev),
                                   Q[0].to(dev), R, 0)
    Kall, Vall = inst_major(K[0]), inst_major(V[0])
    cmp0 = kvr.kvr_get_assignment(sk, 0)[0].reshape(B * H, -1).cpu().numpy()
    cells_o = orc.insert(Kall[:, :N], Vall[:, :N], cmp0, seeds, b)
    ctx = N
    for rnd, n in enumerate(n_new):
        Kr = torch.cat([Kr, K[0, :, :, ctx:ctx + n].to(dev)], dim=2).contiguous()
        Vr = torch.cat([Vr, V[0, :, :, ctx:ctx + n].to(dev)], dim=2).contiguous()
        ret = torch.cat([ret, torch.arange(ctx, ctx + n, dtype=torch.int32, device=dev).expand(B, H, n)], dim=2).contiguous()
        ctx += n
        qd = synth.make_decode_q(2000 + rnd, B, Hq, 128, dtype, dev)
        out = torch.full((B, Hq, 128), float("nan"), dtype=torch.float32, device=dev)
        got = kvr.kvr_decode_attention_static(sk, 0, qd, Kr, Vr, ret, out=out)
        assert kvr.kvr_last_decode_kernel(sk) == kvr.KVR_DECODE_SPLIT
        ordinary = kvr.kvr_decode_attention(sk, 0, qd, Kr, Vr, ret)
        torch.cuda.synchronize()
        want = orc.decode(dec_to_inst(qd, H), inst_major(Kr), inst_major(Vr), ret.reshape(B * H, -1).cpu().numpy(),
                          cells_o, ctx, seeds)
        got_np = got.reshape(B * H, G, 128).cpu().numpy()
        assert np.isfinite(got_np).all()
        assert np.abs(got_np - want).max() <= TOL
        assert (got - ordinary).abs().max().item() <= TOL
    kvr.kvr_sketch_destroy(sk)


def test_static_scratch_decode_rejects_what_does_not_fit():
    """More head-instances than the fixed array has ticket slots for: a clear error, nothing launched."""
    seeds = synth.hash_seeds(92)
    B, H, N = 65, 64, 16                           # 4160 head-instances > 4096
    sk = kvr.kvr_sketch_create(b=1, batch=B, n_layers=1, n_kv_heads=H, n_q_heads=H, max_context=N,
                               kv_dtype=torch.float16, hash_seeds=seeds)
    K, V = synth.make_kv(63, B, H, N, 128, torch.float16, "cuda")
    Q = synth.make_queries(64, B, H, 2, 128, torch.float16, "cuda")
    q = synth.make_decode_q(65, B, H, 128, torch.float16, "cuda")
    Kr, Vr, ret = kvr.kvr_compress(sk, 0, K, V, Q, 4, 0)
    with pytest.raises(kvr.KvrError) as e:
        kvr.kvr_decode_attention_static(sk, 0, q, Kr, Vr, ret)
    assert e.value.status == 7 and "capacity" in str(e.value)
    out = kvr.kvr_decode_attention(sk, 0, q, Kr, Vr, ret)      # the ordinary call still serves this size
    assert torch.isfinite(out).all()
    kvr.kvr_sketch_destroy(sk)
