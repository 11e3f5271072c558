// Host layer of libkvr: handle, argument checks, workspaces and the launch sequences behind the
// C ABI declared in kvr.h.  No arithmetic of the method happens here.
#include <math.h>
#include <new>
#include <string.h>

#include <vector>

#include "kvr_internal.h"

namespace {

#define KVR_CUDA(call)                                 \
    do {                                               \
        cudaError_t e__ = (call);                      \
        if (e__ != cudaSuccess) return map_err(e__);   \
    } while (0)

kvr_status_t map_err(cudaError_t e) {
    if (e == cudaSuccess) return KVR_OK;
    if (e == cudaErrorMemoryAllocation) return KVR_ERR_ALLOC;
    return KVR_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
kvr_status_t dev_alloc(kvr_sketch* sk, T** p, size_t bytes) {
    *p = nullptr;
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes);
    if (e != cudaSuccess) { cudaGetLastError(); *p = nullptr; return KVR_ERR_ALLOC; }
    sk->device_bytes += bytes;
    return KVR_OK;
}

// Grow a workspace; cudaFree orders itself after all work already enqueued on the device.  A workspace
// that has to grow again gets a quarter more than asked for: a generation loop, whose storage grows by
// a row per step, then reallocates (and synchronises the device) once in many steps, not in every one.
kvr_status_t ensure(kvr_sketch* sk, void** p, size_t* cur, size_t need) {
    if (need <= *cur) return KVR_OK;
    const size_t want = *p ? need + need / 4 : need;
    if (*p) { cudaFree(*p); sk->device_bytes -= *cur; *p = nullptr; *cur = 0; }
    need = (need + 255) & ~(size_t)255;
    cudaError_t e = cudaMalloc(p, (want + 255) & ~(size_t)255);
    if (e == cudaSuccess) need = (want + 255) & ~(size_t)255;
    else { cudaGetLastError(); e = cudaMalloc(p, need); }       // no room for the headroom: the exact size
    if (e != cudaSuccess) { cudaGetLastError(); *p = nullptr; return KVR_ERR_ALLOC; }
    *cur = need;
    sk->device_bytes += need;
    return KVR_OK;
}

void free_all(kvr_sketch* sk) {
    void* ptrs[] = {sk->tok_h, sk->tok_g, sk->tok_pack, sk->full_off, sk->full_list, sk->cells, sk->scores,
                    sk->cmp_idx, sk->bitmap, sk->dlist, sk->doff, sk->ws_score, sk->ws_decode, sk->tickets, sk->clist, sk->coff, sk->ctok, sk->dev_status, sk->ml, sk->ws_demote, sk->ws_append, sk->ws_emit,
                    sk->st_K, sk->st_V, sk->st_Q, sk->st_Kr, sk->st_Vr, sk->st_ret, sk->st_q1, sk->st_out};
    for (void* p : ptrs)
        if (p) cudaFree(p);
    if (sk->ev_fork) cudaEventDestroy(sk->ev_fork);
    if (sk->ev_join) cudaEventDestroy(sk->ev_join);
    if (sk->side) cudaStreamDestroy(sk->side);
}

struct LayerRange {
    int inst0, n_inst, layer0, n_layers;
};

kvr_status_t layer_range(const kvr_sketch* sk, int32_t layer, LayerRange* r) {
    if (layer == KVR_ALL_LAYERS) { *r = {0, sk->n_inst, 0, sk->d.n_layers}; return KVR_OK; }
    if (layer < 0 || layer >= sk->d.n_layers) return KVR_ERR_SHAPE;
    *r = {layer * sk->BH, sk->BH, layer, 1};
    return KVR_OK;
}

// Common N / R of the selected layers, or an error when they were not compressed (alike).
kvr_status_t layer_state(const kvr_sketch* sk, const LayerRange& r, int* N, int* R) {
    *N = sk->layer_N[r.layer0];
    *R = sk->layer_R[r.layer0];
    if (*N < 0) return KVR_ERR_STATE;
    for (int l = r.layer0; l < r.layer0 + r.n_layers; ++l)
        if (sk->layer_N[l] != *N || sk->layer_R[l] != *R) return sk->layer_N[l] < 0 ? KVR_ERR_STATE : KVR_ERR_SHAPE;
    return KVR_OK;
}

struct DeviceGuard {
    int prev = -1;
    explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

size_t elem_bytes(const kvr_sketch*) { return 2; }

kvr_status_t compress_impl(kvr_sketch* sk, const LayerRange& lr, const void* K, const void* V, const void* Qobs,
                           int N, int W, int R, int n_recent, void* Kr, void* Vr, int32_t* ret_idx,
                           cudaStream_t st) {
    sk->chain = false;                   // cells and token lists change: the next decode launch waits for everything
    // ---- scores ----
    ScoreShape s;
    s.n_inst = lr.n_inst;
    s.inst0 = lr.inst0;
    s.N = N;
    s.M = sk->G * W;
    s.W = W;
    s.causal = sk->obs_causal;
    s.scale_log2e = (float)(1.4426950408889634 / sqrt((double)sk->d.head_dim));
    const bool tc = sk->score_kernel != KVR_SCORE_MMA_SYNC && kvr_scores_tc_supported(s, K, Qobs);
    if (sk->score_kernel == KVR_SCORE_TCGEN05 && !tc) return KVR_ERR_UNSUPPORTED;
    size_t need;
    if (tc) {
        kvr_scores_tc_plan(sk, &s);
        need = kvr_scores_tc_ws_bytes(s);
    } else {
        int want = (4 * sk->n_sm) / lr.n_inst;
        if (want < 1) want = 1;
        int chunk = (N + want - 1) / want;
        int floor_chunk = N < 256 ? N : 256;
        if (chunk < floor_chunk) chunk = floor_chunk;
        chunk = ((chunk + 63) / 64) * 64;
        s.chunk = chunk;
        s.n_chunks = (N + chunk - 1) / chunk;
        const int Mpad = ((s.M + 127) / 128) * 128;
        need = sizeof(float2) * ((size_t)lr.n_inst * s.n_chunks * Mpad + (size_t)lr.n_inst * Mpad);
    }
    kvr_status_t rc = ensure(sk, &sk->ws_score, &sk->ws_score_bytes, need);
    if (rc != KVR_OK) return rc;
    if (tc) KVR_CUDA(kvr_launch_scores_tc(sk, s, K, Qobs, st));
    else KVR_CUDA(kvr_launch_scores(sk, s, K, Qobs, st));
    sk->last_score_kernel = tc ? KVR_SCORE_TCGEN05 : KVR_SCORE_MMA_SYNC;
    // ---- selection, exact copies, sketch insertion, decode list ----
    // From here on the membership bitmap, the cells and the lists are being rewritten: until every
    // launch below has gone through, the layers count as never compressed (a decode would otherwise
    // read half-written state).
    for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) sk->layer_N[l] = sk->layer_R[l] = -1;
    KVR_CUDA(kvr_launch_select(sk, lr.inst0, lr.n_inst, N, R, n_recent, ret_idx, st));
    // The token lists only need the membership bitmap and a handful of CTAs; they are built on the
    // handle's side stream while the copies and the insertion (thousands of CTAs) run on `st`.
    KVR_CUDA(cudaEventRecord(sk->ev_fork, st));
    KVR_CUDA(cudaStreamWaitEvent(sk->side, sk->ev_fork, 0));
    // The side stream has forked: whatever happens next, it is joined again before this call returns
    // (an unjoined fork would break a stream capture and let the next call race with the lists kernel).
    // (the token lists feed the r = 3 decode kernels; other r walk the compressed-index list)
    cudaError_t e = sk->d.r == KVR_R ? kvr_launch_lists(sk, lr.inst0, lr.n_inst, N, sk->side) : cudaSuccess;
    const cudaError_t e_rec = cudaEventRecord(sk->ev_join, sk->side);
    if (e == cudaSuccess) e = kvr_launch_gather(sk, lr.n_inst, N, R, K, V, ret_idx, Kr, Vr, st);
    if (e == cudaSuccess) e = kvr_launch_insert(sk, lr.inst0, lr.n_inst, N, K, V, st);
    const cudaError_t e_join = (e_rec == cudaSuccess) ? cudaStreamWaitEvent(st, sk->ev_join, 0) : e_rec;
    if (e == cudaSuccess) e = e_join;
    if (e != cudaSuccess) { cudaGetLastError(); return map_err(e); }
    for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) { sk->layer_N[l] = N; sk->layer_R[l] = R; }
    return KVR_OK;
}

// score_acc (or null): also add this call's attention mass to the rows' scores (score_acc) and to the
// vague tokens' scores (the handle's per-token array).
kvr_status_t decode_impl(kvr_sketch* sk, const LayerRange& lr, int N, int R, int rows, const void* q, const void* Kr,
                         const void* Vr, float scale, float* out, cudaStream_t st, float* score_acc = nullptr) {
    if (scale == 0.f) scale = (float)(1.0 / sqrt((double)sk->d.head_dim));
    if (sk->d.r != KVR_R) {                        // r = 1 or 5: the general kernel
        if (sk->decode_kernel == KVR_DECODE_STAGED) return KVR_ERR_UNSUPPORTED;
        const int S = kvr_decode_pick_splits(sk, lr.n_inst, N, R);
        kvr_status_t rc = ensure(sk, &sk->ws_decode, &sk->ws_decode_bytes, kvr_decode_ws_bytes(lr.n_inst, S, sk->G));
        if (rc != KVR_OK) return rc;
        sk->chain = false;
        KVR_CUDA(kvr_launch_decode_generic(sk, lr.inst0, lr.n_inst, N, R, rows, q, Kr, Vr, scale, out, S, st));
        sk->last_decode_kernel = KVR_DECODE_SPLIT;
        return KVR_OK;
    }
    KvrStagedPlan plan;
    if (sk->decode_kernel != KVR_DECODE_SPLIT &&
        kvr_decode_staged_plan(sk, lr.n_inst, N, R, rows, sk->decode_kernel == KVR_DECODE_STAGED, &plan)) {
        kvr_status_t rc = ensure(sk, &sk->ws_decode, &sk->ws_decode_bytes,
                                 kvr_decode_ws_bytes(lr.n_inst, plan.records, sk->G));
        if (rc != KVR_OK) return rc;
        float* emit = nullptr;
        if (score_acc) {                           // the kernel hands out its logits: no second pass over the cache
            rc = ensure(sk, &sk->ws_emit, &sk->ws_emit_bytes,
                        sizeof(float) * (size_t)lr.n_inst * (size_t)(rows + N - R) * sk->G + 16);
            if (rc != KVR_OK) return rc;
            emit = (float*)sk->ws_emit;
        }
        KVR_CUDA(kvr_launch_decode_staged(sk, lr.inst0, lr.n_inst, N, R, rows, q, Kr, Vr, scale, out, plan,
                                          (float*)sk->ws_decode, sk->tickets, emit, st));
        sk->last_decode_kernel = KVR_DECODE_STAGED;
        if (emit) KVR_CUDA(kvr_launch_apply_emitted(sk, lr.inst0, lr.n_inst, rows, N - R, emit, score_acc, st));
        return KVR_OK;
    }
    const int S = kvr_decode_pick_splits(sk, lr.n_inst, N, R);
    kvr_status_t rc = ensure(sk, &sk->ws_decode, &sk->ws_decode_bytes, kvr_decode_ws_bytes(lr.n_inst, S, sk->G));
    if (rc != KVR_OK) return rc;
    KVR_CUDA(kvr_launch_decode(sk, lr.inst0, lr.n_inst, N, R, rows, q, Kr, Vr, scale, out, S, st));
    sk->last_decode_kernel = KVR_DECODE_SPLIT;
    if (score_acc) {                               // the split kernel keeps no logits: a second pass computes them again
        KVR_CUDA(kvr_launch_row_mass(sk, lr.inst0, lr.n_inst, rows, q, Kr, scale, score_acc, st));
        KVR_CUDA(kvr_launch_vague_mass(sk, lr.inst0, lr.n_inst, N - R, q, scale, st));
    }
    return KVR_OK;
}

kvr_status_t check_compress_args(const kvr_sketch* sk, int N, int W, int budget, int n_recent, int* R) {
    if (N < 1 || N > sk->d.max_context || W < 1 || budget < 0 || n_recent < 0) return KVR_ERR_SHAPE;
    if (sk->obs_causal && W > N) return KVR_ERR_SHAPE;       // the window lies inside the context
    *R = budget < N ? budget : N;
    if (n_recent > *R) return KVR_ERR_SHAPE;
    return KVR_OK;
}

}  // namespace

extern "C" {

kvr_status_t kvr_sketch_create(kvr_sketch_t** out, const kvr_sketch_desc_t* desc, const uint32_t* hash_seeds,
                               void* cuda_stream) {
    if (out) *out = nullptr;
    if (!out || !desc || !hash_seeds) return KVR_ERR_INVALID_ARG;
    const kvr_sketch_desc_t& d = *desc;
    if (d.b < 1 || d.n_kv_heads < 1 || d.n_q_heads < 1 || d.batch < 1 || d.n_layers < 1 || d.max_context < 1 ||
        d.r < 1 || d.head_dim < 1)
        return KVR_ERR_INVALID_ARG;
    if (d.kv_dtype != KVR_F16 && d.kv_dtype != KVR_BF16) return KVR_ERR_INVALID_ARG;
    if (d.index_mix != 0 && d.index_mix != 1) return KVR_ERR_INVALID_ARG;
    if (d.n_q_heads % d.n_kv_heads != 0) return KVR_ERR_INVALID_ARG;
    const int G = d.n_q_heads / d.n_kv_heads;
    if ((d.r != 1 && d.r != 3 && d.r != 5) || d.head_dim != KVR_D || d.b > KVR_MAX_B) return KVR_ERR_UNSUPPORTED;
    if (G != 1 && G != 2 && G != 4 && G != 8) return KVR_ERR_UNSUPPORTED;
    const long long n_inst = (long long)d.batch * d.n_layers * d.n_kv_heads;
    if (n_inst > 65535) return KVR_ERR_UNSUPPORTED;
    if (d.seeds_per_head != 0 && d.seeds_per_head != 1) return KVR_ERR_INVALID_ARG;
    const int n_tbl = d.seeds_per_head ? d.n_kv_heads : 1;
    for (int i = 0; i < n_tbl * d.r * 4; ++i)
        if (hash_seeds[i] >= KVR_HASH_P) return KVR_ERR_INVALID_ARG;

    kvr_sketch* sk = new (std::nothrow) kvr_sketch();
    if (!sk) return KVR_ERR_ALLOC;
    sk->d = d;
    sk->G = G;
    sk->BH = d.batch * d.n_kv_heads;
    sk->n_inst = (int)n_inst;
    sk->n_tbl = n_tbl;
    sk->seeds.assign(hash_seeds, hash_seeds + (size_t)n_tbl * d.r * 4);
    sk->layer_N.assign(d.n_layers, -1);
    sk->layer_R.assign(d.n_layers, -1);
    if (cudaGetDevice(&sk->device) != cudaSuccess) { delete sk; return KVR_ERR_CUDA; }
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, sk->device) != cudaSuccess) { delete sk; return KVR_ERR_CUDA; }
    sk->n_sm = prop.multiProcessorCount;
    sk->bitmap_words = (d.max_context + 31) / 32;
    sk->C = d.r == KVR_R ? kvr_decode_staged_pick_C(d.b, G) : 0;
    sk->logC = 0;
    while ((1 << sk->logC) < sk->C) ++sk->logC;
    sk->n1 = sk->C > 0 ? (d.b + sk->C - 1) / sk->C : 0;
    sk->decode_kernel = KVR_DECODE_AUTO;
    sk->wait_ns = 200ull * 1000 * 1000;
    sk->tx_extra = 0;
    sk->last_decode_kernel = KVR_DECODE_AUTO;
    sk->score_kernel = KVR_SCORE_AUTO;
    sk->obs_causal = 0;
    sk->combine = KVR_COMBINE_MEDIAN;
    sk->chain = false;
    sk->chain_stream = nullptr;
    sk->last_score_kernel = KVR_SCORE_AUTO;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (cudaStreamCreateWithFlags(&sk->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&sk->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&sk->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        delete sk;
        return KVR_ERR_CUDA;
    }

    const size_t mc = (size_t)d.max_context, ni = (size_t)n_inst;
    kvr_status_t rc = KVR_OK;
    auto A = [&](auto** p, size_t bytes) { if (rc == KVR_OK) rc = dev_alloc(sk, p, bytes); };
    A(&sk->tok_h, sizeof(int32_t) * n_tbl * d.r * mc);
    A(&sk->tok_g, sizeof(int8_t) * n_tbl * d.r * mc);
    A(&sk->tok_pack, sizeof(uint32_t) * n_tbl * mc);
    A(&sk->full_off, sizeof(int32_t) * n_tbl * d.r * (d.b + 1));
    A(&sk->full_list, sizeof(int32_t) * n_tbl * d.r * mc);
    const size_t cell_bytes = sizeof(float) * ni * 2 * d.r * d.b * KVR_D;
    A(&sk->cells, cell_bytes);
    A(&sk->scores, sizeof(float) * ni * mc);
    A(&sk->cmp_idx, sizeof(int32_t) * ni * mc);
    A(&sk->bitmap, sizeof(uint32_t) * ni * sk->bitmap_words);
    A(&sk->dlist, sizeof(uint32_t) * ni * mc);
    A(&sk->doff, sizeof(int32_t) * ni * (d.b + 1));
    A(&sk->tickets, sizeof(uint32_t) * ni);
    A(&sk->dev_status, sizeof(int32_t));
    A(&sk->ml, sizeof(float) * ni * G * 2);
    if (sk->C > 0) {
        A(&sk->clist, sizeof(uint2) * (ni * mc + 2));     // +2: the staged kernel copies whole 16-byte pairs
        A(&sk->coff, sizeof(int32_t) * ni * (sk->C * sk->C + 1));
        A(&sk->ctok, sizeof(int32_t) * ni * mc);
    }
    if (rc != KVR_OK) { free_all(sk); delete sk; return rc; }
    cudaError_t e = cudaMemsetAsync(sk->cells, 0, cell_bytes, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(sk->tickets, 0, sizeof(uint32_t) * ni, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(sk->dev_status, 0, sizeof(int32_t), st);
    if (e == cudaSuccess && sk->C > 0) e = cudaMemsetAsync(sk->clist, 0, sizeof(uint2) * (ni * mc + 2), st);
    if (e == cudaSuccess && sk->C > 0)
        e = cudaMemsetAsync(sk->coff, 0, sizeof(int32_t) * ni * (sk->C * sk->C + 1), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(sk->doff, 0, sizeof(int32_t) * ni * (d.b + 1), st);
    if (e == cudaSuccess) e = kvr_launch_hash_tables(sk, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) { free_all(sk); delete sk; return map_err(e); }
    *out = sk;
    return KVR_OK;
}

kvr_status_t kvr_sketch_reset(kvr_sketch_t* sk, int32_t layer, void* cuda_stream) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    const size_t per = sizeof(float) * 2 * sk->d.r * sk->d.b * KVR_D;
    sk->chain = false;
    KVR_CUDA(cudaMemsetAsync(sk->cells + (size_t)lr.inst0 * 2 * sk->d.r * sk->d.b * KVR_D, 0, per * lr.n_inst,
                             (cudaStream_t)cuda_stream));
    for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) sk->layer_N[l] = sk->layer_R[l] = -1;
    return KVR_OK;
}

kvr_status_t kvr_sketch_destroy(kvr_sketch_t* sk) {
    if (!sk) return KVR_OK;
    DeviceGuard dg(sk->device);
    cudaDeviceSynchronize();
    free_all(sk);
    delete sk;
    return KVR_OK;
}

size_t kvr_sketch_device_bytes(const kvr_sketch_t* sk) { return sk ? sk->device_bytes : 0; }

int64_t kvr_launch_count(const kvr_sketch_t* sk) { return sk ? sk->launches : 0; }

kvr_status_t kvr_compress(kvr_sketch_t* sk, int32_t layer, const void* K, const void* V, const void* Qobs,
                          int32_t N, int32_t W, int32_t budget, int32_t n_recent, void* Kr, void* Vr,
                          int32_t* ret_idx, void* cuda_stream) {
    if (!sk || !K || !V || !Qobs) return KVR_ERR_INVALID_ARG;
    if (!aligned16(K) || !aligned16(V) || !aligned16(Qobs) || !aligned16(Kr) || !aligned16(Vr) ||
        (reinterpret_cast<uintptr_t>(ret_idx) & 3u))
        return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int R;
    rc = check_compress_args(sk, N, W, budget, n_recent, &R);
    if (rc != KVR_OK) return rc;
    if (R > 0 && (!Kr || !Vr || !ret_idx)) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    return compress_impl(sk, lr, K, V, Qobs, N, W, R, n_recent, Kr, Vr, ret_idx, (cudaStream_t)cuda_stream);
}

kvr_status_t kvr_decode_attention(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr, const void* Vr,
                                  const int32_t* ret_idx, int32_t n_retained, float softmax_scale, float* out,
                                  void* cuda_stream) {
    (void)ret_idx;
    if (!sk || !q || !out) return KVR_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(Kr) || !aligned16(Vr) || !aligned16(out)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_retained < R) return KVR_ERR_SHAPE;          // rows beyond R: tokens appended after the compress
    if (n_retained > 0 && (!Kr || !Vr)) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    return decode_impl(sk, lr, N, R, n_retained, q, Kr, Vr, softmax_scale, out, (cudaStream_t)cuda_stream);
}

kvr_status_t kvr_decode_attention_scored(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr, const void* Vr,
                                         const int32_t* ret_idx, int32_t n_retained, float softmax_scale, float* out,
                                         float* score_acc, void* cuda_stream) {
    (void)ret_idx;
    if (!sk || !q || !out || !score_acc) return KVR_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(Kr) || !aligned16(Vr) || !aligned16(out)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the streaming side is written for r = 3
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_retained < R) return KVR_ERR_SHAPE;
    if (n_retained > 0 && (!Kr || !Vr)) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    return decode_impl(sk, lr, N, R, n_retained, q, Kr, Vr, softmax_scale, out, (cudaStream_t)cuda_stream, score_acc);
}

kvr_status_t kvr_decode_attention_mq(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr, const void* Vr,
                                     const int32_t* ret_idx, int32_t n_retained, int32_t n_queries, int32_t causal,
                                     float softmax_scale, float* out, void* cuda_stream) {
    (void)ret_idx;
    if (!sk || !q || !out) return KVR_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(Kr) || !aligned16(Vr) || !aligned16(out)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale) || (causal != 0 && causal != 1)) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_queries < 1 || n_queries > 4096 || n_retained < R) return KVR_ERR_SHAPE;
    if (causal && n_retained < n_queries) return KVR_ERR_SHAPE;     // the last rows are the queries' own tokens
    if (n_retained > 0 && (!Kr || !Vr)) return KVR_ERR_INVALID_ARG;
    int S, lcap;
    size_t smem;
    if (!kvr_decode_mq_plan(sk, lr.n_inst, N, R, &S, &lcap, &smem)) return KVR_ERR_UNSUPPORTED;
    DeviceGuard dg(sk->device);
    rc = ensure(sk, &sk->ws_decode, &sk->ws_decode_bytes, kvr_decode_mq_ws_bytes(lr.n_inst, sk->C * sk->C * S));
    if (rc != KVR_OK) return rc;
    if (softmax_scale == 0.f) softmax_scale = (float)(1.0 / sqrt((double)sk->d.head_dim));
    sk->chain = false;
    KVR_CUDA(kvr_launch_decode_mq(sk, lr.inst0, lr.n_inst, n_retained, q, Kr, Vr, n_queries, causal, softmax_scale, out, S,
                                  lcap, smem, (float*)sk->ws_decode, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_accumulate_scores(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr, int32_t n_rows,
                                   float softmax_scale, float* score_acc, void* cuda_stream) {
    if (!sk || !q || !score_acc) return KVR_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(Kr)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_rows < 0) return KVR_ERR_SHAPE;
    if (n_rows > 0 && !Kr) return KVR_ERR_INVALID_ARG;
    if (softmax_scale == 0.f) softmax_scale = (float)(1.0 / sqrt((double)sk->d.head_dim));
    DeviceGuard dg(sk->device);
    KVR_CUDA(kvr_launch_row_mass(sk, lr.inst0, lr.n_inst, n_rows, q, Kr, softmax_scale, score_acc,
                                 (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_accumulate_vague_scores(kvr_sketch_t* sk, int32_t layer, const void* q, float softmax_scale,
                                         void* cuda_stream) {
    if (!sk || !q || !aligned16(q)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the streaming side is written for r = 3
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (softmax_scale == 0.f) softmax_scale = (float)(1.0 / sqrt((double)sk->d.head_dim));
    DeviceGuard dg(sk->device);
    KVR_CUDA(kvr_launch_vague_mass(sk, lr.inst0, lr.n_inst, N - R, q, softmax_scale, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_swap(kvr_sketch_t* sk, int32_t layer, void* Kr, void* Vr, int32_t* ret_idx, float* row_scores,
                      int32_t n_rows, int32_t n_recent, float replace_rate, int32_t max_swaps, int32_t* n_swapped,
                      void* cuda_stream) {
    if (!sk || !Kr || !Vr || !ret_idx || !row_scores) return KVR_ERR_INVALID_ARG;
    if (!aligned16(Kr) || !aligned16(Vr)) return KVR_ERR_INVALID_ARG;
    if (!(replace_rate > 0.f) || isinf(replace_rate) || max_swaps < 0) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the streaming side is written for r = 3
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_rows != R || n_recent < 0 || n_recent > n_rows) return KVR_ERR_SHAPE;   // the storage as the last compress / overflow step left it
    DeviceGuard dg(sk->device);
    sk->chain = false;
    KVR_CUDA(kvr_launch_swap(sk, lr.inst0, lr.n_inst, N, N - R, Kr, Vr, ret_idx, row_scores, n_rows, n_recent,
                             replace_rate, max_swaps, n_swapped, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_demote(kvr_sketch_t* sk, int32_t layer, const void* Kr, const void* Vr, const int32_t* ret_idx,
                        const float* row_scores, int32_t n_rows, int32_t new_context, int32_t budget,
                        int32_t n_recent, void* Kr_out, void* Vr_out, int32_t* ret_idx_out, float* row_scores_out,
                        void* cuda_stream) {
    if (!sk || !Kr || !Vr || !ret_idx || !row_scores) return KVR_ERR_INVALID_ARG;
    if (!aligned16(Kr) || !aligned16(Vr) || !aligned16(Kr_out) || !aligned16(Vr_out)) return KVR_ERR_INVALID_ARG;
    if (Kr_out == Kr || Vr_out == Vr || ret_idx_out == ret_idx) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the streaming side is written for r = 3
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (n_rows < R || budget < 0 || budget > n_rows || n_recent < 0 || n_recent > budget) return KVR_ERR_SHAPE;
    // every token that arrived since the last compress / overflow step is one of the rows
    if (new_context > sk->d.max_context || new_context - N != n_rows - R) return KVR_ERR_SHAPE;
    if (budget > 0 && (!Kr_out || !Vr_out || !ret_idx_out)) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    rc = ensure(sk, &sk->ws_demote, &sk->ws_demote_bytes, kvr_demote_ws_bytes(lr.n_inst, n_rows));
    if (rc != KVR_OK) return rc;
    sk->chain = false;
    KVR_CUDA(kvr_launch_demote(sk, lr.inst0, lr.n_inst, n_rows, new_context, budget, n_recent, Kr, Vr, ret_idx,
                               row_scores, Kr_out, Vr_out, ret_idx_out, row_scores_out, sk->ws_demote,
                               (cudaStream_t)cuda_stream));
    for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) { sk->layer_N[l] = new_context; sk->layer_R[l] = budget; }
    return KVR_OK;
}

int32_t kvr_append_sizes(int32_t n_rows, int32_t n_recent, int32_t n_new, int32_t r_budget, int32_t c_budget,
                         int32_t slack, int32_t* n_recent_after) {
    if (n_rows < 0 || n_recent < 0 || n_recent > n_rows || n_new < 0 || r_budget < 0 || c_budget < 0 || slack < 0) return -1;
    long long recent = (long long)n_recent + n_new, cand = (long long)n_rows - n_recent;
    if (recent > (long long)r_budget + slack) { cand += recent - r_budget; recent = r_budget; }
    if (cand > c_budget) cand = c_budget;
    if (cand + recent > 0x7FFFFFFF) return -1;
    if (n_recent_after) *n_recent_after = (int32_t)recent;
    return (int32_t)(cand + recent);
}

kvr_status_t kvr_append(kvr_sketch_t* sk, int32_t layer, const void* Kr, const void* Vr, const int32_t* ret_idx,
                        const float* row_scores, int32_t n_rows, int32_t n_recent, const void* K_new,
                        const void* V_new, int32_t n_new, int32_t r_budget, int32_t c_budget, int32_t slack,
                        float replace_rate, int32_t max_swaps, void* Kr_out, void* Vr_out, int32_t* ret_idx_out,
                        float* row_scores_out, int32_t* n_swapped, void* cuda_stream) {
    if (!sk || !Kr_out || !Vr_out || !ret_idx_out || !row_scores_out) return KVR_ERR_INVALID_ARG;
    if (n_rows > 0 && (!Kr || !Vr || !ret_idx || !row_scores)) return KVR_ERR_INVALID_ARG;
    if (n_new > 0 && (!K_new || !V_new)) return KVR_ERR_INVALID_ARG;
    if (!aligned16(Kr) || !aligned16(Vr) || !aligned16(K_new) || !aligned16(V_new) || !aligned16(Kr_out) || !aligned16(Vr_out))
        return KVR_ERR_INVALID_ARG;
    if (Kr_out == Kr || Vr_out == Vr || ret_idx_out == ret_idx || row_scores_out == row_scores) return KVR_ERR_INVALID_ARG;
    if (!(replace_rate > 0.f) || isinf(replace_rate) || max_swaps < 0) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the streaming side is written for r = 3
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    int32_t recent_after = 0;
    const int32_t rows_after = kvr_append_sizes(n_rows, n_recent, n_new, r_budget, c_budget, slack, &recent_after);
    if (rows_after < 0 || n_rows < R) return KVR_ERR_SHAPE;
    const int rows_cat = n_rows + n_new;
    const int ctx0 = N + (n_rows - R);                     // every token that arrived since the last compress / overflow step is a row
    if (ctx0 + n_new > sk->d.max_context) return KVR_ERR_SHAPE;
    DeviceGuard dg(sk->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const bool pops = rows_after < rows_cat;               // known from the counts alone: no device result is waited for
    if (!pops) {
        KVR_CUDA(kvr_launch_append_rows(sk, lr.n_inst, Kr, Vr, ret_idx, row_scores, n_rows, K_new, V_new, n_new, ctx0,
                                        Kr_out, Vr_out, ret_idx_out, row_scores_out, st));
    } else {
        // storage + new rows go to a workspace; the overflow step compacts them into the caller's output
        const size_t row_b = (size_t)KVR_D * 2;
        const size_t per = (size_t)lr.n_inst * rows_cat;
        const size_t off_v = (per * row_b + 255) & ~(size_t)255, off_r = off_v + ((per * row_b + 255) & ~(size_t)255);
        const size_t off_s = off_r + ((per * 4 + 255) & ~(size_t)255), total = off_s + per * 4;
        rc = ensure(sk, &sk->ws_append, &sk->ws_append_bytes, total);
        if (rc != KVR_OK) return rc;
        rc = ensure(sk, &sk->ws_demote, &sk->ws_demote_bytes, kvr_demote_ws_bytes(lr.n_inst, rows_cat));
        if (rc != KVR_OK) return rc;
        char* w = (char*)sk->ws_append;
        KVR_CUDA(kvr_launch_append_rows(sk, lr.n_inst, Kr, Vr, ret_idx, row_scores, n_rows, K_new, V_new, n_new, ctx0,
                                        w, w + off_v, (int32_t*)(w + off_r), (float*)(w + off_s), st));
        sk->chain = false;
        for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) sk->layer_N[l] = sk->layer_R[l] = -1;
        KVR_CUDA(kvr_launch_demote(sk, lr.inst0, lr.n_inst, rows_cat, ctx0 + n_new, rows_after, recent_after, w, w + off_v,
                                   (const int32_t*)(w + off_r), (const float*)(w + off_s), Kr_out, Vr_out, ret_idx_out,
                                   row_scores_out, sk->ws_demote, st));
        N = ctx0 + n_new;
        R = rows_after;
        for (int l = lr.layer0; l < lr.layer0 + lr.n_layers; ++l) { sk->layer_N[l] = N; sk->layer_R[l] = R; }
    }
    // the swap loop runs on every call (Algorithm 3), on the device, over what the steps above left
    if (rows_after - recent_after > 0 && N - R > 0 && max_swaps > 0) {
        sk->chain = false;
        KVR_CUDA(kvr_launch_swap(sk, lr.inst0, lr.n_inst, N, N - R, Kr_out, Vr_out, ret_idx_out, row_scores_out, rows_after,
                                 recent_after, replace_rate, max_swaps, n_swapped, st));
    } else if (n_swapped) {
        KVR_CUDA(cudaMemsetAsync(n_swapped, 0, sizeof(int32_t) * lr.n_inst, st));
    }
    return KVR_OK;
}

kvr_status_t kvr_compress_host(kvr_sketch_t* sk, int32_t layer, const void* K, const void* V, const void* Qobs,
                               int32_t N, int32_t W, int32_t budget, int32_t n_recent, void* cuda_stream) {
    if (!sk || !K || !V || !Qobs) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int R;
    rc = check_compress_args(sk, N, W, budget, n_recent, &R);
    if (rc != KVR_OK) return rc;
    DeviceGuard dg(sk->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t kv_bytes = (size_t)lr.n_inst * N * KVR_D * elem_bytes(sk);
    const size_t q_bytes = (size_t)lr.n_inst * sk->G * W * KVR_D * elem_bytes(sk);
    // staging for the inputs of this call
    rc = ensure(sk, &sk->st_K, &sk->st_k_bytes, kv_bytes);
    if (rc == KVR_OK) rc = ensure(sk, &sk->st_V, &sk->st_v_bytes, kv_bytes);
    if (rc == KVR_OK) rc = ensure(sk, &sk->st_Q, &sk->st_q_bytes, q_bytes);
    if (rc != KVR_OK) return rc;
    // handle-owned store of the retained rows: one fixed row count for all layers
    if (!sk->st_Kr && R > 0) {
        const size_t rows = (size_t)sk->n_inst * R;
        rc = dev_alloc(sk, (char**)&sk->st_Kr, rows * KVR_D * elem_bytes(sk));
        if (rc == KVR_OK) rc = dev_alloc(sk, (char**)&sk->st_Vr, rows * KVR_D * elem_bytes(sk));
        if (rc == KVR_OK) rc = dev_alloc(sk, &sk->st_ret, rows * sizeof(int32_t));
        if (rc != KVR_OK) return rc;
        sk->st_ret_rows = (size_t)R;
    }
    if (R > 0 && (size_t)R != sk->st_ret_rows) return KVR_ERR_SHAPE;
    KVR_CUDA(cudaMemcpyAsync(sk->st_K, K, kv_bytes, cudaMemcpyHostToDevice, st));
    KVR_CUDA(cudaMemcpyAsync(sk->st_V, V, kv_bytes, cudaMemcpyHostToDevice, st));
    KVR_CUDA(cudaMemcpyAsync(sk->st_Q, Qobs, q_bytes, cudaMemcpyHostToDevice, st));
    const size_t row0 = (size_t)lr.inst0 * R;
    char* Kr = R > 0 ? (char*)sk->st_Kr + row0 * KVR_D * elem_bytes(sk) : nullptr;
    char* Vr = R > 0 ? (char*)sk->st_Vr + row0 * KVR_D * elem_bytes(sk) : nullptr;
    int32_t* ret = R > 0 ? sk->st_ret + row0 : nullptr;
    rc = compress_impl(sk, lr, sk->st_K, sk->st_V, sk->st_Q, N, W, R, n_recent, Kr, Vr, ret, st);
    if (rc != KVR_OK) return rc;
    KVR_CUDA(cudaStreamSynchronize(st));   // the caller may reuse its host buffers
    return KVR_OK;
}

kvr_status_t kvr_decode_attention_host(kvr_sketch_t* sk, int32_t layer, const void* q, float softmax_scale,
                                       float* out, void* cuda_stream) {
    if (!sk || !q || !out) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (R > 0 && (!sk->st_Kr || (size_t)R != sk->st_ret_rows)) return KVR_ERR_STATE;
    DeviceGuard dg(sk->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t q_bytes = (size_t)lr.n_inst * sk->G * KVR_D * elem_bytes(sk);
    const size_t o_bytes = (size_t)lr.n_inst * sk->G * KVR_D * sizeof(float);
    rc = ensure(sk, &sk->st_q1, &sk->st_q1_bytes, q_bytes);
    if (rc == KVR_OK) rc = ensure(sk, &sk->st_out, &sk->st_out_bytes, o_bytes);
    if (rc != KVR_OK) return rc;
    KVR_CUDA(cudaMemcpyAsync(sk->st_q1, q, q_bytes, cudaMemcpyHostToDevice, st));
    const size_t row0 = (size_t)lr.inst0 * R;
    const char* Kr = R > 0 ? (const char*)sk->st_Kr + row0 * KVR_D * elem_bytes(sk) : nullptr;
    const char* Vr = R > 0 ? (const char*)sk->st_Vr + row0 * KVR_D * elem_bytes(sk) : nullptr;
    rc = decode_impl(sk, lr, N, R, R, sk->st_q1, Kr, Vr, softmax_scale, (float*)sk->st_out, st);
    if (rc != KVR_OK) return rc;
    KVR_CUDA(cudaMemcpyAsync(out, sk->st_out, o_bytes, cudaMemcpyDeviceToHost, st));
    KVR_CUDA(cudaStreamSynchronize(st));
    return KVR_OK;
}

kvr_status_t kvr_get_scores(const kvr_sketch_t* sk, int32_t layer, float* s, void* cuda_stream) {
    if (!sk || !s) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    DeviceGuard dg(sk->device);
    KVR_CUDA(cudaMemcpy2DAsync(s, sizeof(float) * N, sk->scores + (size_t)lr.inst0 * sk->d.max_context,
                               sizeof(float) * sk->d.max_context, sizeof(float) * N, lr.n_inst,
                               cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_get_assignment(const kvr_sketch_t* sk, int32_t layer, int32_t* cmp_idx, int32_t* bucket,
                                int8_t* sign, void* cuda_stream) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    DeviceGuard dg(sk->device);
    KVR_CUDA(kvr_launch_assignment(sk, lr.inst0, lr.n_inst, N - R, cmp_idx, bucket, sign, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_get_cells(const kvr_sketch_t* sk, int32_t layer, float* cells, void* cuda_stream) {
    if (!sk || !cells) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    DeviceGuard dg(sk->device);
    const size_t per = (size_t)2 * sk->d.r * sk->d.b * KVR_D;
    KVR_CUDA(cudaMemcpyAsync(cells, sk->cells + (size_t)lr.inst0 * per, sizeof(float) * per * lr.n_inst,
                             cudaMemcpyDeviceToDevice, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_reconstruct(const kvr_sketch_t* sk, int32_t layer, float* Kt, float* Vt, void* cuda_stream) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    if (!aligned16(Kt) || !aligned16(Vt)) return KVR_ERR_INVALID_ARG;
    LayerRange lr;
    kvr_status_t rc = layer_range(sk, layer, &lr);
    if (rc != KVR_OK) return rc;
    int N, R;
    rc = layer_state(sk, lr, &N, &R);
    if (rc != KVR_OK) return rc;
    if (N == R) return KVR_OK;   // nothing was compressed: empty outputs
    if (!Kt && !Vt) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    if (sk->d.r != KVR_R) KVR_CUDA(kvr_launch_reconstruct_generic(sk, lr.inst0, lr.n_inst, N - R, Kt, Vt, (cudaStream_t)cuda_stream));
    else KVR_CUDA(kvr_launch_reconstruct(sk, lr.inst0, lr.n_inst, N - R, Kt, Vt, (cudaStream_t)cuda_stream));
    return KVR_OK;
}

kvr_status_t kvr_sketch_set_decode_kernel(kvr_sketch_t* sk, int32_t which) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    if (which != KVR_DECODE_AUTO && which != KVR_DECODE_SPLIT && which != KVR_DECODE_STAGED) return KVR_ERR_INVALID_ARG;
    sk->decode_kernel = which;
    return KVR_OK;
}

kvr_status_t kvr_sketch_device_status(kvr_sketch_t* sk, int32_t* status, void* cuda_stream) {
    if (!sk || !status) return KVR_ERR_INVALID_ARG;
    DeviceGuard dg(sk->device);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    KVR_CUDA(cudaMemcpyAsync(status, sk->dev_status, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    KVR_CUDA(cudaStreamSynchronize(st));
    return KVR_OK;
}

kvr_status_t kvr_sketch_set_wait_test(kvr_sketch_t* sk, int64_t wait_limit_ns, int32_t unannounced_bytes) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    // the copies land within microseconds: a limit of 100 us or more never cuts a copy short
    if (wait_limit_ns < 100 * 1000 || wait_limit_ns > 1000ll * 1000 * 1000) return KVR_ERR_INVALID_ARG;
    if (unannounced_bytes < 0 || unannounced_bytes > 4096 || (unannounced_bytes & 15)) return KVR_ERR_INVALID_ARG;
    sk->wait_ns = (unsigned long long)wait_limit_ns;
    sk->tx_extra = (uint32_t)unannounced_bytes;
    return KVR_OK;
}

int32_t kvr_last_decode_kernel(const kvr_sketch_t* sk) { return sk ? sk->last_decode_kernel : KVR_DECODE_AUTO; }

kvr_status_t kvr_sketch_set_score_kernel(kvr_sketch_t* sk, int32_t which) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    if (which != KVR_SCORE_AUTO && which != KVR_SCORE_MMA_SYNC && which != KVR_SCORE_TCGEN05) return KVR_ERR_INVALID_ARG;
    sk->score_kernel = which;
    return KVR_OK;
}

kvr_status_t kvr_paper_storage_split(int32_t context, float ratio, int32_t* exact_rows, int32_t* n_recent, int32_t* b) {
    if (context < 1 || !(ratio > 0.f) || ratio > 1.f || !exact_rows || !n_recent || !b) return KVR_ERR_INVALID_ARG;
    const int total = (int)floor((double)ratio * context + 0.5);
    int cells = (int)floor(0.1 * total / KVR_R + 0.5);
    if (cells < 1) cells = 1;
    int exact = total - KVR_R * cells;
    if (exact < 0) exact = 0;
    *b = cells;
    *exact_rows = exact;
    *n_recent = exact / 2;
    return KVR_OK;
}

kvr_status_t kvr_layer_budgets(const double* weights, int32_t n_layers, int32_t context, float ratio,
                               int32_t* budgets) {
    if (!weights || !budgets || n_layers < 1 || context < 1 || !(ratio > 0.f) || ratio > 1.f) return KVR_ERR_INVALID_ARG;
    double wsum = 0.0;
    for (int l = 0; l < n_layers; ++l) {
        if (!(weights[l] >= 0.0) || isinf(weights[l])) return KVR_ERR_INVALID_ARG;
        wsum += weights[l];
    }
    if (!(wsum > 0.0)) return KVR_ERR_INVALID_ARG;
    const long long mean = (long long)floor((double)ratio * context + 0.5);
    long long total = mean * n_layers;
    std::vector<double> share(n_layers, 0.0);
    std::vector<char> full(n_layers, 0);
    // proportional shares; a layer that would exceed the context is capped and the rest re-shared
    double left = (double)total, wleft = wsum;
    for (int round = 0; round < n_layers; ++round) {
        bool capped = false;
        for (int l = 0; l < n_layers; ++l) {
            if (full[l]) continue;
            if (wleft > 0.0 && left * weights[l] / wleft > (double)context) {
                full[l] = 1;
                share[l] = (double)context;
                capped = true;
            }
        }
        if (!capped) break;
        left = (double)total;
        wleft = 0.0;
        for (int l = 0; l < n_layers; ++l) {
            if (full[l]) left -= (double)context;
            else wleft += weights[l];
        }
        if (left < 0.0) left = 0.0;
    }
    long long given = 0;
    for (int l = 0; l < n_layers; ++l) {
        if (!full[l]) share[l] = wleft > 0.0 ? left * weights[l] / wleft : 0.0;
        budgets[l] = (int32_t)floor(share[l]);
        given += budgets[l];
    }
    // largest remainder, lower layer first among equals
    long long target = total;
    if (target > (long long)n_layers * context) target = (long long)n_layers * context;
    while (given < target) {
        int best = -1;
        double best_frac = -1.0;
        for (int l = 0; l < n_layers; ++l) {
            if (budgets[l] >= context) continue;
            const double frac = share[l] - floor(share[l]);
            if (frac > best_frac) { best_frac = frac; best = l; }
        }
        if (best < 0) break;
        budgets[best] += 1;
        share[best] = floor(share[best]);      // its remainder is used up
        given += 1;
    }
    return KVR_OK;
}

kvr_status_t kvr_sketch_set_combine(kvr_sketch_t* sk, int32_t which) {
    if (!sk || (which != KVR_COMBINE_MEDIAN && which != KVR_COMBINE_MEAN)) return KVR_ERR_INVALID_ARG;
    sk->combine = which;
    return KVR_OK;
}

kvr_status_t kvr_sketch_set_obs_window_causal(kvr_sketch_t* sk, int32_t on) {
    if (!sk || (on != 0 && on != 1)) return KVR_ERR_INVALID_ARG;
    sk->obs_causal = on;
    return KVR_OK;
}

int32_t kvr_last_score_kernel(const kvr_sketch_t* sk) { return sk ? sk->last_score_kernel : KVR_SCORE_AUTO; }

kvr_status_t kvr_layer_shape(const kvr_sketch_t* sk, int32_t layer, int32_t* N, int32_t* R) {
    if (!sk) return KVR_ERR_INVALID_ARG;
    if (layer < 0 || layer >= sk->d.n_layers) return KVR_ERR_SHAPE;
    if (sk->layer_N[layer] < 0) return KVR_ERR_STATE;
    if (N) *N = sk->layer_N[layer];
    if (R) *R = sk->layer_R[layer];
    return KVR_OK;
}

const char* kvr_status_string(kvr_status_t st) {
    switch (st) {
        case KVR_OK: return "ok";
        case KVR_ERR_INVALID_ARG: return "invalid argument";
        case KVR_ERR_UNSUPPORTED: return "unsupported configuration";
        case KVR_ERR_SHAPE: return "shape mismatch";
        case KVR_ERR_ALLOC: return "device allocation failed";
        case KVR_ERR_CUDA: return "CUDA error";
        case KVR_ERR_STATE: return "layer not compressed";
        case KVR_ERR_LIMIT: return "built-in capacity exceeded";
    }
    return "unknown status";
}

}  // extern "C"
