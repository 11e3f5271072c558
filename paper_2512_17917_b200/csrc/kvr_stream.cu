// Streaming side of Algorithm 3 (Compress on an existing storage):
//   * attention mass of the exactly stored rows under the softmax of the last decode (the paper ranks
//     tokens by accumulated attention scores, "the result of Softmax(QK^T)", Overview);
//   * the overflow step: when the exact storage (Recent + Candidate) holds more rows than its budget,
//     the newest n_recent rows stay, the best-scored of the others stay, and every other row is
//     handed to the Vague sketch with Algorithm 1 (added to the existing cells: insertion is linear).
//   * the attention mass of the reconstructed (Vague) tokens, added to the handle's per-token scores;
//   * the swap loop: while the worst candidate's score times ReplaceRate is below the best vague
//     token's score, that token is queried (Algorithm 2), deleted from the sketch (Algorithm 1 with the
//     negated vectors), the candidate inserted in its place, and the queried vectors stored as the
//     candidate's row.
// Selection reuses the top-k kernel of the one-shot compress on the row scores; the per-token lists the
// decode kernels walk are rebuilt from the updated membership bitmap.
#include "kvr_internal.h"

namespace {

template <typename T>
__device__ __forceinline__ void unpack8(const uint4& x, float (&f)[8]) {
    float2 a = KvrType<T>::to_f2(x.x), b = KvrType<T>::to_f2(x.y), c = KvrType<T>::to_f2(x.z),
           d = KvrType<T>::to_f2(x.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

// One half-warp per stored row: mass = sum_g 2^(q_g . k scale log2e - M_g) / L_g with (M_g, L_g) the
// reference maximum and sum the layer's last decode left for this head-instance.
template <typename T, int G>
__global__ void __launch_bounds__(256)
row_mass_kernel(const uint4* __restrict__ q, const uint4* __restrict__ Kr, const float* __restrict__ ml_all,
                int inst0, int rows, float scale_log2e, float* __restrict__ acc) {
    const int u = blockIdx.y, inst = inst0 + u;
    const int row = blockIdx.x * 16 + (threadIdx.x >> 4), l16 = threadIdx.x & 15;
    const bool ok = row < rows;
    float kf[8];
    unpack8<T>(Kr[((size_t)u * rows + (ok ? row : 0)) * 16 + l16], kf);
    float mass = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        float qf[8];
        unpack8<T>(q[((size_t)u * G + g) * 16 + l16], qf);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
        for (int off = 8; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        const float M = ml_all[((size_t)inst * G + g) * 2], L = ml_all[((size_t)inst * G + g) * 2 + 1];
        mass += exp2f(s * scale_log2e - M) / L;
    }
    if (ok && l16 == 0) acc[(size_t)u * rows + row] += mass;
}

// One warp per compressed token: keys only of Algorithm 2 (element-wise median of its three cells),
// logits against the G queries, mass under the (maximum, sum) the layer's last decode left.
template <typename T, int G>
__global__ void __launch_bounds__(256)
vague_mass_kernel(const uint2* __restrict__ q, const float* __restrict__ cells_all, const int32_t* __restrict__ cmp_all,
                  const int32_t* __restrict__ tok_h, const float* __restrict__ ml_all, int max_ctx, int b, int a,
                  int inst0, int n_tbl, int mean, float scale_log2e, float* __restrict__ scores_all) {
    const int u = blockIdx.y, inst = inst0 + u, lane = threadIdx.x & 31;
    tok_h += (size_t)(n_tbl > 1 ? inst % n_tbl : 0) * KVR_R * max_ctx;
    const int t = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (t >= a) return;                                           // (whole warp)
    const int J = cmp_all[(size_t)inst * max_ctx + t];
    const float* ck = cells_all + (size_t)inst * 2 * KVR_R * b * KVR_D;
    float4 k[KVR_R];
#pragma unroll
    for (int i = 0; i < KVR_R; ++i)
        k[i] = *reinterpret_cast<const float4*>(ck + ((size_t)i * b + tok_h[(size_t)i * max_ctx + J]) * KVR_D + 4 * lane);
    const float kx = kvr_comb3(k[0].x, k[1].x, k[2].x, mean), ky = kvr_comb3(k[0].y, k[1].y, k[2].y, mean);
    const float kz = kvr_comb3(k[0].z, k[1].z, k[2].z, mean), kw = kvr_comb3(k[0].w, k[1].w, k[2].w, mean);
    float mass = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint2 qq = q[((size_t)u * G + g) * 32 + lane];
        const float2 q0 = KvrType<T>::to_f2(qq.x), q1 = KvrType<T>::to_f2(qq.y);
        float s = fmaf(q0.x, kx, fmaf(q0.y, ky, fmaf(q1.x, kz, q1.y * kw)));
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        const float M = ml_all[((size_t)inst * G + g) * 2], L = ml_all[((size_t)inst * G + g) * 2 + 1];
        mass += exp2f(s * scale_log2e - M) / L;
    }
    if (lane == 0) scores_all[(size_t)inst * max_ctx + J] += mass;
}

// The same two sums from logits a decode kernel already computed (the staged kernel writes them out on
// request): one thread per logit slot; slot < rows is a retained row, the others are class-list entries,
// whose token indices the list builder recorded.  No pass over the cache.
template <int G>
__global__ void __launch_bounds__(256)
apply_emitted_kernel(const float* __restrict__ emit, const float* __restrict__ ml_all, const int32_t* __restrict__ ctok_all,
                     int rows, int a, int max_ctx, int inst0, float* __restrict__ acc, float* __restrict__ scores_all) {
    const int u = blockIdx.y, inst = inst0 + u;
    const int slot = blockIdx.x * 256 + threadIdx.x;
    if (slot >= rows + a) return;
    const float* e = emit + ((size_t)u * (rows + a) + slot) * G;
    float x[G];
    if constexpr (G == 4) { const float4 v = *reinterpret_cast<const float4*>(e); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
    else if constexpr (G == 2) { const float2 v = *reinterpret_cast<const float2*>(e); x[0] = v.x; x[1] = v.y; }
    else x[0] = e[0];
    float mass = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float M = ml_all[((size_t)inst * G + g) * 2], L = ml_all[((size_t)inst * G + g) * 2 + 1];
        mass += exp2f(x[g] - M) / L;
    }
    if (slot < rows) acc[(size_t)u * rows + slot] += mass;
    else scores_all[(size_t)inst * max_ctx + ctok_all[(size_t)inst * max_ctx + (slot - rows)]] += mass;
}

__device__ __forceinline__ uint32_t swap_score_key(float s) {      // order-preserving integer image of a float
    const uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
template <bool MAX>
__device__ __forceinline__ unsigned long long swap_block_reduce(unsigned long long v, unsigned long long* s_w, int lane,
                                                                int warp) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long x = __shfl_xor_sync(0xFFFFFFFFu, v, o);
        v = MAX ? (x > v ? x : v) : (x < v ? x : v);
    }
    if (lane == 0) s_w[warp] = v;
    __syncthreads();
    unsigned long long r = s_w[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long x = __shfl_xor_sync(0xFFFFFFFFu, r, o);
        r = MAX ? (x > r ? x : r) : (x < r ? x : r);
    }
    __syncthreads();
    return r;                                                     // the same value in every thread
}

// ---- the swap loop of Algorithm 3, one CTA of 1024 threads per head-instance ------------------------
// Candidate part = rows [0, rows - n_recent); Vague part = the `a` tokens listed in cmp (their scores
// in the handle's per-token array).  Equal scores: the lower token index is taken, for the minimum
// and for the maximum.  The decision C.Min * ReplaceRate < V.Max is taken in fp32.
struct SwapArgs {
    int32_t* ret; float* rs; float* scores; int32_t* cmp; uint32_t* bitmap; float* cK; float* cV;
    const int32_t* tok_h; const int8_t* tok_g;
    int n_cand, a, max_ctx, b, mean;
    float rate;
};
__device__ __forceinline__ unsigned long long swap_cand_key(const SwapArgs& A, int r) {      // smallest = worst candidate
    return ((unsigned long long)swap_score_key(A.rs[r]) << 32) | (uint32_t)A.ret[r];
}
__device__ __forceinline__ unsigned long long swap_vague_key(const SwapArgs& A, int t) {     // smallest = best vague token
    const int J = A.cmp[t];
    return ((unsigned long long)(~swap_score_key(A.scores[J])) << 32) | (uint32_t)J;
}

// One swap, by threads 0..255 (keys | values x channel) and one bookkeeping thread; the caller
// synchronises before (the pair is read by everybody) and after.
template <typename T>
__device__ __forceinline__ void swap_one(const SwapArgs& A, T* Kr, T* Vr, int row, int pos, int tid) {
    const int Jc = A.ret[row], Jv = A.cmp[pos];
    const float c_min = A.rs[row], v_max = A.scores[Jv];
    __syncthreads();                                          // everybody has read the pair before it is rewritten
    if (tid < 2 * KVR_D) {
        const int d = tid & (KVR_D - 1);
        const bool val = tid >= KVR_D;
        float* cells = val ? A.cV : A.cK;
        T* rowp = (val ? Vr : Kr) + (size_t)row * KVR_D + d;
        float x[KVR_R], g[KVR_R];
        size_t cell[KVR_R];
#pragma unroll
        for (int i = 0; i < KVR_R; ++i) {
            cell[i] = ((size_t)i * A.b + A.tok_h[(size_t)i * A.max_ctx + Jv]) * KVR_D + d;
            g[i] = val ? (float)A.tok_g[(size_t)i * A.max_ctx + Jv] : 1.f;
            x[i] = g[i] * cells[cell[i]];
        }
        const float m = kvr_comb3(x[0], x[1], x[2], A.mean);        // query the vague token (Algorithm 2)
#pragma unroll
        for (int i = 0; i < KVR_R; ++i) cells[cell[i]] -= g[i] * m; // take it out of the sketch again
        const float c = KvrType<T>::to_float(*rowp);
#pragma unroll
        for (int i = 0; i < KVR_R; ++i) {                           // the candidate's vectors go in (Algorithm 1)
            const size_t cc = ((size_t)i * A.b + A.tok_h[(size_t)i * A.max_ctx + Jc]) * KVR_D + d;
            cells[cc] += (val ? (float)A.tok_g[(size_t)i * A.max_ctx + Jc] : 1.f) * c;
        }
        *rowp = KvrType<T>::from_float(m);                          // the queried vectors take its row
    }
    if (tid == 1023) {
        A.ret[row] = Jv;
        A.rs[row] = v_max;
        A.scores[Jc] = c_min;
        A.cmp[pos] = Jc;
        atomicOr(&A.bitmap[Jv >> 5], 1u << (Jv & 31));
        atomicAnd(&A.bitmap[Jc >> 5], ~(1u << (Jc & 31)));
    }
}

// The loop as the algorithm prints it: find the pair, decide, swap, again.
template <typename T>
__device__ int swap_loop_in_order(const SwapArgs& A, T* Kr, T* Vr, int done, int max_swaps, unsigned long long* s_w, int* s_pair) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (; done < max_swaps; ++done) {
        unsigned long long best = ~0ull;
        int best_i = -1;
        for (int r = tid; r < A.n_cand; r += 1024) {
            const unsigned long long key = swap_cand_key(A, r);
            if (key < best) { best = key; best_i = r; }
        }
        const unsigned long long cmin = swap_block_reduce<false>(best, s_w, lane, warp);
        if (best_i >= 0 && best == cmin) s_pair[0] = best_i;
        best = ~0ull;
        best_i = -1;
        for (int t = tid; t < A.a; t += 1024) {
            const unsigned long long key = swap_vague_key(A, t);
            if (key < best) { best = key; best_i = t; }
        }
        const unsigned long long vmax = swap_block_reduce<false>(best, s_w, lane, warp);
        if (best_i >= 0 && best == vmax) s_pair[1] = best_i;
        __syncthreads();
        const int row = s_pair[0], pos = s_pair[1];
        if (!(__fmul_rn(A.rs[row], A.rate) < A.scores[A.cmp[pos]])) break;      // (uniform)
        swap_one<T>(A, Kr, Vr, row, pos, tid);
        __syncthreads();                                          // the next round sees this one's writes
    }
    return done;
}

// The K smallest of n distinct 64-bit keys (hi(i) << 32 | lo(i)), ascending: their positions go to
// out_pos[0..K).  All 1024 threads call it.  hi(i) is cheap (the caller keeps the score images in
// shared memory where they fit); lo(i) reads global memory.
//   1. Every thread takes the smallest high word of its own keys (i = tid, tid + 1024, ...); a value U
//      with at least K of these 1024 minima at or below it bounds the K-th key from above, because K
//      different keys lie at or below it.
//   2. The keys with high word <= U are collected (normally a small multiple of K) and sorted.
//   3. Should they not fit (more than SW_M: many equal scores), the K-th key is found bit by bit
//      instead: T grows from the top bit down while fewer than K keys lie below it, one count over
//      all keys per bit; then the same among the low words of the keys that share T.
constexpr int SW_K = 256, SW_M = 2048;
__device__ __forceinline__ int swap_block_sum(int v, int* s_cnt) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    if (lane == 0) s_cnt[warp] = v;
    __syncthreads();
    int t = s_cnt[lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
    __syncthreads();
    return t;                                                     // the same value in every thread
}
template <class HiFn, class LoFn>
__device__ void swap_select(int n, int K, HiFn hi, LoFn lo, unsigned long long* s_lk, int* s_lp, int* s_cnt, int* s_misc,
                            int* out_pos) {
    const int tid = threadIdx.x, lane = tid & 31;
    // ---- 1. a bound from the threads' minima: every warp sorts its 32 minima (shuffles only) and names its
    // t-th smallest, t = ceil(K / 32); the largest of the 32 warps' answers has at least 32 t >= K keys at or
    // below it.  (One barrier instead of a bit-by-bit search for the exact K-th minimum; a little looser.)
    uint32_t U;
    {
        uint32_t mn = 0xFFFFFFFFu;
        for (int i = tid; i < n; i += 1024) mn = min(mn, hi(i));
        if (tid == 0) s_misc[2] = 0;
#pragma unroll
        for (int k = 2; k <= 32; k <<= 1)
#pragma unroll
            for (int j = k >> 1; j > 0; j >>= 1) {
                const uint32_t o = __shfl_xor_sync(0xFFFFFFFFu, mn, j);
                const bool up = ((lane & k) == 0) == ((lane & j) == 0);      // this lane keeps the smaller of the two
                mn = up ? min(mn, o) : max(mn, o);
            }
        const int t = (K + 31) >> 5;                              // 1 .. SW_K / 32
        const uint32_t mine = __shfl_sync(0xFFFFFFFFu, mn, t - 1);
        if (lane == 0) s_cnt[tid >> 5] = (int)mine;
        __syncthreads();
        uint32_t v = (uint32_t)s_cnt[lane];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xFFFFFFFFu, v, o));
        U = v;
        __syncthreads();
    }
    // ---- 2. the keys at or below U (a warp reserves its places with one addition)
    for (int base = 0; base < n; base += 1024) {
        const int i = base + tid;
        uint32_t h = 0u;
        const bool in = i < n && (h = hi(i)) <= U;
        const unsigned m = __ballot_sync(0xFFFFFFFFu, in);
        int at = 0;
        if (lane == 0 && m) at = atomicAdd(&s_misc[2], __popc(m));
        at = __shfl_sync(0xFFFFFFFFu, at, 0) + __popc(m & ((1u << lane) - 1u));
        if (in && at < SW_M) {
            s_lk[at] = ((unsigned long long)h << 32) | lo(i);
            s_lp[at] = i;
        }
    }
    __syncthreads();
    int M = s_misc[2];
    __syncthreads();
    if (M > SW_M) {
        // ---- 3. too many: find the K-th key bit by bit and collect up to it
        uint32_t T = 0u;
        int less = 0;                                             // keys whose high word is below T
        for (int bit = 31; bit >= 0; --bit) {
            const uint32_t trial = T | (1u << bit);
            int c = 0;
            for (int i = tid; i < n; i += 1024) c += hi(i) < trial ? 1 : 0;
            c = swap_block_sum(c, s_cnt);
            if (c < K) { T = trial; less = c; }
        }
        int ties = 0;
        for (int i = tid; i < n; i += 1024) ties += hi(i) == T ? 1 : 0;
        ties = swap_block_sum(ties, s_cnt);
        uint32_t TL = 0xFFFFFFFFu;
        const int need = K - less;                                // of the `ties` keys with high word T
        if (ties > need) {
            TL = 0u;
            for (int bit = 31; bit >= 0; --bit) {
                const uint32_t trial = TL | (1u << bit);
                int c = 0;
                for (int i = tid; i < n; i += 1024)
                    if (hi(i) == T) c += lo(i) < trial ? 1 : 0;
                c = swap_block_sum(c, s_cnt);
                if (c < need) TL = trial;
            }
        }
        if (tid == 0) s_misc[2] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += 1024) {
            const uint32_t h = hi(i);
            if (h <= T) {
                const uint32_t l = lo(i);
                if (h < T || l <= TL) {
                    const int at = atomicAdd(&s_misc[2], 1);
                    if (at < SW_M) {                              // (keys that are not distinct would give more than K)
                        s_lk[at] = ((unsigned long long)h << 32) | l;
                        s_lp[at] = i;
                    }
                }
            }
        }
        __syncthreads();
        M = min(s_misc[2], SW_M);
        __syncthreads();
    }
    int P = 32;
    while (P < M) P <<= 1;
    for (int i = M + tid; i < P; i += 1024) { s_lk[i] = ~0ull; s_lp[i] = 0; }
    __syncthreads();
    if (P <= 1024) {
        // one key per thread: exchanges between lanes of a warp go through shuffles, the others through
        // shared memory with a barrier (10 of the 45 steps of a sort of 512)
        unsigned long long key = tid < P ? s_lk[tid] : ~0ull;
        int pos = tid < P ? s_lp[tid] : 0;
        for (int k = 2; k <= P; k <<= 1)
            for (int j = k >> 1; j > 0; j >>= 1) {
                unsigned long long ok;
                int op;
                if (j >= 32) {
                    __syncthreads();                              // (everybody has read the previous exchange)
                    if (tid < P) { s_lk[tid] = key; s_lp[tid] = pos; }
                    __syncthreads();
                    ok = tid < P ? s_lk[tid ^ j] : ~0ull;
                    op = tid < P ? s_lp[tid ^ j] : 0;
                } else {
                    ok = __shfl_xor_sync(0xFFFFFFFFu, key, j);
                    op = __shfl_xor_sync(0xFFFFFFFFu, pos, j);
                }
                const bool keep_small = ((tid & k) == 0) == ((tid & j) == 0);
                if (keep_small ? ok < key : ok > key) { key = ok; pos = op; }
            }
        __syncthreads();
        if (tid < P) { s_lk[tid] = key; s_lp[tid] = pos; }
        __syncthreads();
    } else {
        for (int k = 2; k <= P; k <<= 1)
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int i = tid; i < P; i += 1024) {
                    const int x = i ^ j;
                    if (x > i) {
                        const unsigned long long ka = s_lk[i], kb = s_lk[x];
                        if ((ka > kb) == ((i & k) == 0)) {
                            s_lk[i] = kb; s_lk[x] = ka;
                            const int pa = s_lp[i]; s_lp[i] = s_lp[x]; s_lp[x] = pa;
                        }
                    }
                }
                __syncthreads();
            }
    }
    if (tid < K) out_pos[tid] = s_lp[tid];
    __syncthreads();
}

// With ReplaceRate >= 1 and scores >= 0 the loop never touches a token twice: a token that has just
// become a candidate scores more than the minimum it replaced times the rate, so once it is the
// minimum the test fails; a token that has just become vague scores less than the maximum it
// replaced, so once it is the maximum the test fails as well.  The k-th swap therefore pairs the
// k-th worst candidate with the k-th best vague token of the lists as they stand at entry, up to
// the first pair that fails the test: both lists are selected and sorted in parallel (up to SW_K
// pairs per round), and only the updates of the cells, which do depend on their order, run one
// after the other, without any search in between.  Other rates or scores take the loop in order.
template <typename T>
__global__ void __launch_bounds__(1024)
swap_kernel(T* __restrict__ Kr_all, T* __restrict__ Vr_all, int32_t* __restrict__ ret_all, float* __restrict__ rs_all,
            int rows, int n_recent, float rate, int max_swaps, float* __restrict__ scores_all,
            int32_t* __restrict__ cmp_all, int a, uint32_t* __restrict__ bitmap_all, int bitmap_words,
            float* __restrict__ cells_all, const int32_t* __restrict__ tok_h, const int8_t* __restrict__ tok_g,
            int max_ctx, int b, int inst0, int n_tbl, int mean, int n_cache, int32_t* __restrict__ n_swapped) {
    extern __shared__ uint32_t s_img[];                          // score images of the first n_cache candidates, then vague tokens
    __shared__ unsigned long long s_w[32];
    __shared__ unsigned long long s_lk[SW_M];                    // scratch of the selection: keys, positions
    __shared__ int s_lp[SW_M];
    __shared__ int s_posC[SW_K], s_posV[SW_K], s_Jc[SW_K], s_Jv[SW_K];
    __shared__ float s_c[SW_K], s_v[SW_K];
    __shared__ uint16_t s_hC[SW_K][KVR_R], s_hV[SW_K][KVR_R];     // cell index | sign bit << 15
    __shared__ int s_cnt[32], s_misc[4], s_pair[2], s_nsw;
    const int u = blockIdx.x, inst = inst0 + u, tid = threadIdx.x;
    SwapArgs A;
    A.tok_h = tok_h + (size_t)(n_tbl > 1 ? inst % n_tbl : 0) * KVR_R * max_ctx;
    A.tok_g = tok_g + (size_t)(n_tbl > 1 ? inst % n_tbl : 0) * KVR_R * max_ctx;
    T* Kr = Kr_all + (size_t)u * rows * KVR_D;
    T* Vr = Vr_all + (size_t)u * rows * KVR_D;
    A.ret = ret_all + (size_t)u * rows;
    A.rs = rs_all + (size_t)u * rows;
    A.scores = scores_all + (size_t)inst * max_ctx;
    A.cmp = cmp_all + (size_t)inst * max_ctx;
    A.bitmap = bitmap_all + (size_t)inst * bitmap_words;
    A.cK = cells_all + (size_t)inst * 2 * KVR_R * b * KVR_D;
    A.cV = A.cK + (size_t)KVR_R * b * KVR_D;
    A.n_cand = rows - n_recent;
    A.a = a; A.max_ctx = max_ctx; A.b = b; A.mean = mean; A.rate = rate;
    int done = 0;
    if (A.n_cand > 0 && a > 0 && max_swaps > 0) {
        // a score with its sign bit set, or a rate below one: the argument above does not hold
        int odd = !(rate >= 1.f);
        const int nc_c = min(A.n_cand, n_cache), nc_v = min(a, n_cache - nc_c);
        for (int r = tid; r < A.n_cand; r += 1024) {
            const float sc = A.rs[r];
            odd |= (int)(__float_as_uint(sc) >> 31);
            if (r < nc_c) s_img[r] = swap_score_key(sc);
        }
        for (int t = tid; t < a; t += 1024) {
            const float sc = A.scores[A.cmp[t]];
            odd |= (int)(__float_as_uint(sc) >> 31);
            if (t < nc_v) s_img[nc_c + t] = ~swap_score_key(sc);
        }
        odd = __syncthreads_or(odd);
        if (odd) {
            done = swap_loop_in_order<T>(A, Kr, Vr, 0, max_swaps, s_w, s_pair);
        } else {
            for (;;) {
                const int K = min(min(max_swaps - done, SW_K), min(A.n_cand, a));
                swap_select(A.n_cand, K, [&](int r) { return r < nc_c ? s_img[r] : swap_score_key(A.rs[r]); },
                            [&](int r) { return (uint32_t)A.ret[r]; }, s_lk, s_lp, s_cnt, s_misc, s_posC);
                swap_select(a, K, [&](int t) { return t < nc_v ? s_img[nc_c + t] : ~swap_score_key(A.scores[A.cmp[t]]); },
                            [&](int t) { return (uint32_t)A.cmp[t]; }, s_lk, s_lp, s_cnt, s_misc, s_posV);
                if (tid == 0) s_nsw = K;
                __syncthreads();
                if (tid < K) {
                    const int row = s_posC[tid], pos = s_posV[tid];
                    const int Jc = A.ret[row], Jv = A.cmp[pos];
                    const float c = A.rs[row], v = A.scores[Jv];
                    s_Jc[tid] = Jc; s_Jv[tid] = Jv; s_c[tid] = c; s_v[tid] = v;
#pragma unroll
                    for (int i = 0; i < KVR_R; ++i) {
                        s_hC[tid][i] = (uint16_t)(A.tok_h[(size_t)i * max_ctx + Jc] | (A.tok_g[(size_t)i * max_ctx + Jc] < 0 ? 0x8000 : 0));
                        s_hV[tid][i] = (uint16_t)(A.tok_h[(size_t)i * max_ctx + Jv] | (A.tok_g[(size_t)i * max_ctx + Jv] < 0 ? 0x8000 : 0));
                    }
                    if (!(__fmul_rn(c, rate) < v)) atomicMin(&s_nsw, tid);          // the loop ends at the first such pair
                }
                __syncthreads();
                const int n_sw = s_nsw;
                if (tid < 2 * KVR_D) {                            // the cells and the rows, swap after swap
                    const int d = tid & (KVR_D - 1);
                    const bool val = tid >= KVR_D;
                    float* cells = (val ? A.cV : A.cK) + d;
                    T* rowsp = (val ? Vr : Kr) + d;
                    for (int k = 0; k < n_sw; ++k) {
                        // everything the swap reads is asked for at once (one round trip to memory per swap);
                        // where the candidate's cell is the vague token's own, it takes the value just computed
                        float xv[KVR_R], xc[KVR_R], gv[KVR_R], gc[KVR_R];
                        size_t cv[KVR_R], cc[KVR_R];
                        T* rp = rowsp + (size_t)s_posC[k] * KVR_D;
#pragma unroll
                        for (int i = 0; i < KVR_R; ++i) {
                            const uint32_t ev = s_hV[k][i], ec = s_hC[k][i];
                            cv[i] = ((size_t)i * b + (ev & 0x7FFFu)) * KVR_D;
                            cc[i] = ((size_t)i * b + (ec & 0x7FFFu)) * KVR_D;
                            gv[i] = (val && (ev & 0x8000u)) ? -1.f : 1.f;
                            gc[i] = (val && (ec & 0x8000u)) ? -1.f : 1.f;
                            xv[i] = cells[cv[i]];
                            xc[i] = cells[cc[i]];
                        }
                        const float c = KvrType<T>::to_float(*rp);
                        const float m = kvr_comb3(gv[0] * xv[0], gv[1] * xv[1], gv[2] * xv[2], mean);    // Algorithm 2
#pragma unroll
                        for (int i = 0; i < KVR_R; ++i) {
                            const float nv = xv[i] - gv[i] * m;               // the vague token leaves the sketch
                            const float nc = (cc[i] == cv[i] ? nv : xc[i]) + gc[i] * c;              // the candidate enters it (Algorithm 1)
                            cells[cv[i]] = nv;
                            cells[cc[i]] = nc;
                        }
                        *rp = KvrType<T>::from_float(m);
                    }
                } else {                                          // who is where, and with which score
                    for (int k = tid - 2 * KVR_D; k < n_sw; k += 1024 - 2 * KVR_D) {
                        const int row = s_posC[k], pos = s_posV[k], Jc = s_Jc[k], Jv = s_Jv[k];
                        A.ret[row] = Jv;
                        A.rs[row] = s_v[k];
                        A.scores[Jc] = s_c[k];
                        A.cmp[pos] = Jc;
                        if (row < nc_c) s_img[row] = swap_score_key(s_v[k]);
                        if (pos < nc_v) s_img[nc_c + pos] = ~swap_score_key(s_c[k]);
                        atomicOr(&A.bitmap[Jv >> 5], 1u << (Jv & 31));
                        atomicAnd(&A.bitmap[Jc >> 5], ~(1u << (Jc & 31)));
                    }
                }
                done += n_sw;
                __syncthreads();
                if (n_sw < K || K < SW_K || done >= max_swaps) break;
            }
        }
    }
    if (tid == 0 && n_swapped) n_swapped[u] = done;
}

// Bookkeeping of the overflow step: kept rows -> compacted index / score lists and membership bits
// set; evicted rows -> membership bits cleared and their token indices listed for the insertion.
__global__ void demote_tokens_kernel(const int32_t* __restrict__ keep_pos, const int32_t* __restrict__ evict_pos,
                                     const int32_t* __restrict__ ret_idx, const float* __restrict__ scores,
                                     int rows, int budget, int inst0, uint32_t* __restrict__ bitmap_all,
                                     int bitmap_words, int32_t* __restrict__ ret_out, float* __restrict__ scores_out,
                                     int32_t* __restrict__ ev_tok, float* __restrict__ tok_scores_all, int max_ctx) {
    const int u = blockIdx.y, i = blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t* bitmap = bitmap_all + (size_t)(inst0 + u) * bitmap_words;
    if (i < budget) {
        const int pos = keep_pos[(size_t)u * budget + i];
        const int J = ret_idx[(size_t)u * rows + pos];
        ret_out[(size_t)u * budget + i] = J;
        if (scores_out) scores_out[(size_t)u * budget + i] = scores[(size_t)u * rows + pos];
        atomicOr(&bitmap[J >> 5], 1u << (J & 31));
    }
    if (i < rows - budget) {
        const int pos = evict_pos[(size_t)u * rows + i];
        const int J = ret_idx[(size_t)u * rows + pos];
        ev_tok[(size_t)u * rows + i] = J;
        tok_scores_all[(size_t)(inst0 + u) * max_ctx + J] = scores[(size_t)u * rows + pos];   // V.Max_Score reads it
        atomicAnd(&bitmap[J >> 5], ~(1u << (J & 31)));
    }
}

// Algorithm 1 for the evicted rows, added to the existing cells.  One CTA per (cell, row, instance)
// walks the evicted list in order (ascending token index) and sums its own tokens with a
// compensated accumulator: no atomics, bit-reproducible.
template <typename T>
__global__ void __launch_bounds__(128)
insert_rows_kernel(const int32_t* __restrict__ tok_h, const int8_t* __restrict__ tok_g,
                   const int32_t* __restrict__ ev_tok, const int32_t* __restrict__ evict_pos,
                   const uint32_t* __restrict__ Kr, const uint32_t* __restrict__ Vr, int rows, int n_ev, int max_ctx,
                   int b, int inst0, int n_tbl, float* __restrict__ cells_all) {
    const int c = blockIdx.x, i = blockIdx.y, u = blockIdx.z, inst = inst0 + u;
    tok_h += (size_t)(n_tbl > 1 ? inst % n_tbl : 0) * KVR_R * max_ctx;
    tok_g += (size_t)(n_tbl > 1 ? inst % n_tbl : 0) * KVR_R * max_ctx;
    const int tid = threadIdx.x, half = tid >> 6, c2 = tid & 63;
    const int32_t* h = tok_h + (size_t)i * max_ctx;
    const int8_t* g = tok_g + (size_t)i * max_ctx;
    const uint32_t* src = (half ? Vr : Kr) + (size_t)u * rows * (KVR_D / 2) + c2;
    float sx = 0.f, sy = 0.f, cx = 0.f, cy = 0.f;
    bool any = false;
    for (int t = 0; t < n_ev; ++t) {
        const int J = ev_tok[(size_t)u * rows + t];
        if (h[J] != c) continue;
        any = true;
        float2 f = KvrType<T>::to_f2(src[(size_t)evict_pos[(size_t)u * rows + t] * (KVR_D / 2)]);
        if (half && g[J] < 0) { f.x = -f.x; f.y = -f.y; }
        float s = sx + f.x;
        cx += (fabsf(sx) >= fabsf(f.x)) ? (sx - s) + f.x : (f.x - s) + sx;
        sx = s;
        s = sy + f.y;
        cy += (fabsf(sy) >= fabsf(f.y)) ? (sy - s) + f.y : (f.y - s) + sy;
        sy = s;
    }
    if (!any) return;
    float2* cell = reinterpret_cast<float2*>(cells_all + ((((size_t)inst * 2 + half) * KVR_R + i) * b + c) * KVR_D + 2 * c2);
    float2 v = *cell;
    v.x += sx + cx;
    v.y += sy + cy;
    *cell = v;
}

// Ascending list of the compressed tokens (index < N, membership bit clear) of one head-instance:
// a thread takes 32 tokens (one bitmap word) at a time, the CTA scans the counts.
__global__ void __launch_bounds__(1024)
cmp_from_bitmap_kernel(const uint32_t* __restrict__ bitmap_all, int bitmap_words, int N, int max_ctx, int inst0,
                       int32_t* __restrict__ cmp_all) {
    __shared__ int s_warp[32];
    __shared__ int s_run;
    const int inst = inst0 + blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t* bitmap = bitmap_all + (size_t)inst * bitmap_words;
    int32_t* cmp = cmp_all + (size_t)inst * max_ctx;
    const int words = (N + 31) >> 5;
    if (tid == 0) s_run = 0;
    __syncthreads();
    for (int base = 0; base < words; base += 1024) {
        const int w = base + tid;
        uint32_t out = 0u;                                        // bit set = compressed token
        if (w < words) {
            out = ~bitmap[w];
            if (w == words - 1 && (N & 31)) out &= (1u << (N & 31)) - 1u;
        }
        const int n = __popc(out);
        int inc = n;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
            if (lane >= o) inc += t;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        int wsum = s_warp[lane], winc = wsum;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xFFFFFFFFu, winc, o);
            if (lane >= o) winc += t;
        }
        const int before_warp = __shfl_sync(0xFFFFFFFFu, winc - wsum, warp);
        const int total = __shfl_sync(0xFFFFFFFFu, winc, 31);
        const int at = s_run + before_warp + inc - n;
        for (int l = 0; l < 32; ++l) {                            // word by word: a warp writes neighbouring entries
            const uint32_t m = __shfl_sync(0xFFFFFFFFu, out, l);
            const int at_l = __shfl_sync(0xFFFFFFFFu, at, l);
            if ((m >> lane) & 1u) cmp[at_l + __popc(m & ((1u << lane) - 1u))] = ((base + (warp << 5) + l) << 5) + lane;
        }
        __syncthreads();
        if (tid == 0) s_run += total;
        __syncthreads();
    }
}

// Storage of a head-instance followed by the newly arrived rows (Algorithm 3 pushes new tokens to the
// Recent part, which is the tail of the storage): rows, token indices (the new tokens are numbered
// ctx0, ctx0 + 1, ...) and row scores (a new token has received no attention yet: 0).
__global__ void append_rows_kernel(const uint4* __restrict__ Kr, const uint4* __restrict__ Vr,
                                   const int32_t* __restrict__ ret, const float* __restrict__ rs, int rows,
                                   const uint4* __restrict__ Kn, const uint4* __restrict__ Vn, int n_new, int ctx0,
                                   uint4* __restrict__ Ko, uint4* __restrict__ Vo, int32_t* __restrict__ ro,
                                   float* __restrict__ so) {
    const int u = blockIdx.y, total = rows + n_new;
    constexpr int RV = KVR_D * 2 / 16;                        // 16-byte pieces of a 16-bit row
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total * RV; i += gridDim.x * blockDim.x) {
        const int row = i / RV, c = i - row * RV;
        const bool old = row < rows;
        const size_t src = old ? ((size_t)u * rows + row) * RV + c : ((size_t)u * n_new + (row - rows)) * RV + c;
        Ko[((size_t)u * total + row) * RV + c] = old ? Kr[src] : Kn[src];
        Vo[((size_t)u * total + row) * RV + c] = old ? Vr[src] : Vn[src];
    }
    for (int row = blockIdx.x * blockDim.x + threadIdx.x; row < total; row += gridDim.x * blockDim.x) {
        ro[(size_t)u * total + row] = row < rows ? ret[(size_t)u * rows + row] : ctx0 + (row - rows);
        so[(size_t)u * total + row] = row < rows ? rs[(size_t)u * rows + row] : 0.f;
    }
}

}  // namespace

cudaError_t kvr_launch_append_rows(kvr_sketch* sk, int n_inst, const void* Kr, const void* Vr, const int32_t* ret,
                                   const float* rs, int rows, const void* Kn, const void* Vn, int n_new, int ctx0,
                                   void* Ko, void* Vo, int32_t* ro, float* so, cudaStream_t st) {
    if (rows + n_new <= 0 || n_inst <= 0) return cudaSuccess;
    const int total = rows + n_new;
    int gx = (total * 16 + 255) / 256;
    if (gx > 64) gx = 64;
    append_rows_kernel<<<dim3(gx, n_inst), 256, 0, st>>>((const uint4*)Kr, (const uint4*)Vr, ret, rs, rows, (const uint4*)Kn,
                                                         (const uint4*)Vn, n_new, ctx0, (uint4*)Ko, (uint4*)Vo, ro, so);
    sk->launches += 1;
    return cudaGetLastError();
}

cudaError_t kvr_launch_row_mass(kvr_sketch* sk, int inst0, int n_inst, int rows, const void* q, const void* Kr,
                                float scale, float* acc, cudaStream_t st) {
    if (rows <= 0) return cudaSuccess;
    const dim3 grid((rows + 15) / 16, n_inst);
    const float sl = scale * 1.4426950408889634f;
    const bool f16 = sk->d.kv_dtype == KVR_F16;
#define KVR_RM(TT, GG) row_mass_kernel<TT, GG><<<grid, 256, 0, st>>>((const uint4*)q, (const uint4*)Kr, sk->ml, inst0, rows, sl, acc)
    switch (sk->G) {
        case 1: if (f16) KVR_RM(__half, 1); else KVR_RM(__nv_bfloat16, 1); break;
        case 2: if (f16) KVR_RM(__half, 2); else KVR_RM(__nv_bfloat16, 2); break;
        case 4: if (f16) KVR_RM(__half, 4); else KVR_RM(__nv_bfloat16, 4); break;
        case 8: if (f16) KVR_RM(__half, 8); else KVR_RM(__nv_bfloat16, 8); break;
        default: return cudaErrorInvalidValue;
    }
#undef KVR_RM
    sk->launches += 1;
    return cudaGetLastError();
}

cudaError_t kvr_launch_vague_mass(kvr_sketch* sk, int inst0, int n_inst, int a, const void* q, float scale,
                                  cudaStream_t st) {
    if (a <= 0) return cudaSuccess;
    const dim3 grid((a + 7) / 8, n_inst);
    const float sl = scale * 1.4426950408889634f;
    const bool f16 = sk->d.kv_dtype == KVR_F16;
#define KVR_VM(TT, GG) vague_mass_kernel<TT, GG><<<grid, 256, 0, st>>>((const uint2*)q, sk->cells, sk->cmp_idx, sk->tok_h, sk->ml, sk->d.max_context, sk->d.b, a, inst0, sk->n_tbl, sk->combine, sl, sk->scores)
    switch (sk->G) {
        case 1: if (f16) KVR_VM(__half, 1); else KVR_VM(__nv_bfloat16, 1); break;
        case 2: if (f16) KVR_VM(__half, 2); else KVR_VM(__nv_bfloat16, 2); break;
        case 4: if (f16) KVR_VM(__half, 4); else KVR_VM(__nv_bfloat16, 4); break;
        case 8: if (f16) KVR_VM(__half, 8); else KVR_VM(__nv_bfloat16, 8); break;
        default: return cudaErrorInvalidValue;
    }
#undef KVR_VM
    sk->launches += 1;
    return cudaGetLastError();
}

cudaError_t kvr_launch_apply_emitted(kvr_sketch* sk, int inst0, int n_inst, int rows, int a, const float* emit,
                                     float* score_acc, cudaStream_t st) {
    if (rows + a <= 0) return cudaSuccess;
    const dim3 grid((rows + a + 255) / 256, n_inst);
    switch (sk->G) {
        case 1: apply_emitted_kernel<1><<<grid, 256, 0, st>>>(emit, sk->ml, sk->ctok, rows, a, sk->d.max_context, inst0, score_acc, sk->scores); break;
        case 2: apply_emitted_kernel<2><<<grid, 256, 0, st>>>(emit, sk->ml, sk->ctok, rows, a, sk->d.max_context, inst0, score_acc, sk->scores); break;
        case 4: apply_emitted_kernel<4><<<grid, 256, 0, st>>>(emit, sk->ml, sk->ctok, rows, a, sk->d.max_context, inst0, score_acc, sk->scores); break;
        default: return cudaErrorInvalidValue;
    }
    sk->launches += 1;
    return cudaGetLastError();
}

// The swap loop, then the compressed-token list and the decode lists rebuilt from the bitmap.
cudaError_t kvr_launch_swap(kvr_sketch* sk, int inst0, int n_inst, int N, int a, void* Kr, void* Vr, int32_t* ret_idx,
                            float* row_scores, int rows, int n_recent, float rate, int max_swaps, int32_t* n_swapped,
                            cudaStream_t st) {
    const int mc = sk->d.max_context;
    // shared memory for the score images of candidates and vague tokens, as many as fit
    const int n_cache = std::min(std::max(rows - n_recent, 0) + a, (int)((160 * 1024) / sizeof(uint32_t)));
    const size_t smem = sizeof(uint32_t) * (size_t)std::max(n_cache, 1);
    cudaError_t e0 = cudaSuccess;
    if (sk->d.kv_dtype == KVR_F16) {
        e0 = cudaFuncSetAttribute(swap_kernel<__half>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e0 != cudaSuccess) return e0;
        swap_kernel<__half><<<n_inst, 1024, smem, st>>>((__half*)Kr, (__half*)Vr, ret_idx, row_scores, rows, n_recent, rate,
                                                        max_swaps, sk->scores, sk->cmp_idx, a, sk->bitmap, sk->bitmap_words,
                                                        sk->cells, sk->tok_h, sk->tok_g, mc, sk->d.b, inst0, sk->n_tbl,
                                                        sk->combine, n_cache, n_swapped);
    } else {
        e0 = cudaFuncSetAttribute(swap_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e0 != cudaSuccess) return e0;
        swap_kernel<__nv_bfloat16><<<n_inst, 1024, smem, st>>>((__nv_bfloat16*)Kr, (__nv_bfloat16*)Vr, ret_idx, row_scores,
                                                               rows, n_recent, rate, max_swaps, sk->scores, sk->cmp_idx, a,
                                                               sk->bitmap, sk->bitmap_words, sk->cells, sk->tok_h,
                                                               sk->tok_g, mc, sk->d.b, inst0, sk->n_tbl, sk->combine,
                                                               n_cache, n_swapped);
    }
    cmp_from_bitmap_kernel<<<n_inst, 1024, 0, st>>>(sk->bitmap, sk->bitmap_words, N, mc, inst0, sk->cmp_idx);
    sk->launches += 2;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return kvr_launch_lists(sk, inst0, n_inst, N, st);
}

// workspace: keep_pos [n][rows], evict_pos [n][rows], ev_tok [n][rows] (int32), row bitmap [n][ceil(rows/32)]
size_t kvr_demote_ws_bytes(int n_inst, int rows) {
    return sizeof(int32_t) * (size_t)n_inst * ((size_t)3 * rows + (rows + 31) / 32 + 4);
}

cudaError_t kvr_launch_demote(kvr_sketch* sk, int inst0, int n_inst, int rows, int N_new, int budget, int n_recent,
                              const void* Kr, const void* Vr, const int32_t* ret_idx, const float* row_scores,
                              void* Kr_out, void* Vr_out, int32_t* ret_out, float* scores_out, void* ws,
                              cudaStream_t st) {
    int32_t* keep_pos = (int32_t*)ws;
    int32_t* evict_pos = keep_pos + (size_t)n_inst * rows;
    int32_t* ev_tok = evict_pos + (size_t)n_inst * rows;
    uint32_t* row_bits = (uint32_t*)(ev_tok + (size_t)n_inst * rows);
    const int words_r = (rows + 31) / 32, n_ev = rows - budget, b = sk->d.b, mc = sk->d.max_context;
    // which rows stay: the top-k rule of the one-shot compress applied to the row scores
    cudaError_t e = kvr_launch_select_rows(sk, row_scores, rows, n_inst, budget, n_recent, keep_pos, evict_pos,
                                           row_bits, words_r, st);
    if (e != cudaSuccess) return e;
    if (budget > 0) {
        e = kvr_launch_gather(sk, n_inst, rows, budget, Kr, Vr, keep_pos, Kr_out, Vr_out, st);
        if (e != cudaSuccess) return e;
    }
    demote_tokens_kernel<<<dim3((rows + 255) / 256, n_inst), 256, 0, st>>>(
        keep_pos, evict_pos, ret_idx, row_scores, rows, budget, inst0, sk->bitmap, sk->bitmap_words, ret_out,
        scores_out, ev_tok, sk->scores, mc);
    if (n_ev > 0) {
        const dim3 g(b, KVR_R, n_inst);
        if (sk->d.kv_dtype == KVR_F16)
            insert_rows_kernel<__half><<<g, 128, 0, st>>>(sk->tok_h, sk->tok_g, ev_tok, evict_pos, (const uint32_t*)Kr,
                                                          (const uint32_t*)Vr, rows, n_ev, mc, b, inst0, sk->n_tbl, sk->cells);
        else
            insert_rows_kernel<__nv_bfloat16><<<g, 128, 0, st>>>(sk->tok_h, sk->tok_g, ev_tok, evict_pos,
                                                                 (const uint32_t*)Kr, (const uint32_t*)Vr, rows, n_ev,
                                                                 mc, b, inst0, sk->n_tbl, sk->cells);
    }
    cmp_from_bitmap_kernel<<<n_inst, 1024, 0, st>>>(sk->bitmap, sk->bitmap_words, N_new, mc, inst0, sk->cmp_idx);
    sk->launches += 2 + (n_ev > 0 ? 1 : 0);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    return kvr_launch_lists(sk, inst0, n_inst, N_new, st);
}
