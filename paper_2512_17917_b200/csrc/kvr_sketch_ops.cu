// Vague-sketch insertion (Algorithm 1) and the stand-alone query (Algorithm 2).
//
// Insertion is a deterministic segmented reduction keyed by cell: one CTA owns one cell of one
// row of one head-instance, walks that cell's token list (ascending token index, built once per
// handle from the hash tables), skips retained tokens by the membership bitmap, and adds
//     cell.key += K[J],     cell.value += g_i(J) * V[J]
// in fp32: the tokens of the list are dealt to four half-warps in turn, each summing its own in ascending
// order (batches of eight rows added plainly, the batch sums accumulated with compensation), and the
// four sums are added in a fixed order at the end.  No atomics: the cells are bit-reproducible.
#include "kvr_internal.h"

namespace {

constexpr int INS_THREADS = 128;   // warp w: keys (w even) or values (w odd); its two half-warps and the two warps of a kind take every fourth token each
constexpr int INS_UNROLL = 8;      // rows requested per lane before the first is added

template <typename T>
__global__ void __launch_bounds__(INS_THREADS)
insert_kernel(const int32_t* __restrict__ full_off, const int32_t* __restrict__ full_list,
              const int8_t* __restrict__ tok_g, const uint32_t* __restrict__ bitmap_all, int bitmap_words,
              const uint4* __restrict__ K, const uint4* __restrict__ V, int N, int max_ctx, int b,
              int inst0, int n_tbl, int r, float* __restrict__ cells_all) {
    __shared__ uint32_t s_tok[INS_THREADS];
    __shared__ int s_wcnt[INS_THREADS / 32];
    __shared__ float4 s_part[2][KVR_D / 4];      // sums of the tokens 2, 3 (mod 4): [keys | values][4 channels]

    const int c = blockIdx.x, i = blockIdx.y, u = blockIdx.z, inst = inst0 + u;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, l16 = lane & 15;
    const int kv = warp & 1, par = (warp >> 1) * 2 + (lane >> 4);             // this half-warp's tokens: par, par + 4, ...
    const uint32_t* bitmap = bitmap_all + (size_t)inst * bitmap_words;
    const int tb = n_tbl > 1 ? inst % n_tbl : 0;              // hash tables of this kv head (seeds per head) or the shared ones
    full_off += (size_t)tb * r * (b + 1);
    const int32_t* list = full_list + ((size_t)tb * r + i) * max_ctx;
    const int8_t* g = tok_g + ((size_t)tb * r + i) * max_ctx;
    const uint4* src = (kv ? V : K) + (size_t)u * N * (KVR_D / 8) + l16;      // 8 channels (16 bytes) per lane
    const int p0 = full_off[i * (b + 1) + c], p1 = full_off[i * (b + 1) + c + 1];
    kvr_pdl_trigger();
    kvr_pdl_wait();            // (as a dependent of the kernel before it: the membership bitmap is complete from here on)

    // Two levels: the rows of one batch (up to INS_UNROLL) are added plainly, in order, and the batch
    // sum goes into a compensated running sum, so the rounding error does not grow with the length
    // of the cell's token list.
    float s[8], cc[8], blk[8];
#pragma unroll
    for (int d = 0; d < 8; ++d) s[d] = cc[d] = blk[d] = 0.f;
    auto add = [&](const uint4& x, uint32_t e) {
        const float sg = (kv && (e >> 31)) ? -1.f : 1.f;      // g_i(J) for the values, +1 for the keys
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 f = KvrType<T>::to_f2(w[q]);
            blk[2 * q] = fmaf(f.x, sg, blk[2 * q]);           // = blk + g v, rounded once
            blk[2 * q + 1] = fmaf(f.y, sg, blk[2 * q + 1]);
        }
    };
    auto fold = [&]() {
#pragma unroll
        for (int d = 0; d < 8; ++d) {
            const float v = blk[d], t = s[d] + v;
            cc[d] += (fabsf(s[d]) >= fabsf(v)) ? (s[d] - t) + v : (v - t) + s[d];
            s[d] = t;
        }
    };

    for (int base = p0; base < p1; base += INS_THREADS) {
        const int p = base + tid;
        bool keep = false;
        uint32_t packed = 0;
        if (p < p1) {
            int J = list[p];
            if (J < N && !((bitmap[J >> 5] >> (J & 31)) & 1u)) {
                keep = true;
                packed = (uint32_t)J | ((g[J] < 0) ? 0x80000000u : 0u);
            }
        }
        unsigned m = __ballot_sync(0xFFFFFFFFu, keep);
        if (lane == 0) s_wcnt[warp] = __popc(m);
        __syncthreads();
        int off = 0, n = 0;
#pragma unroll
        for (int w = 0; w < INS_THREADS / 32; ++w) {
            if (w < warp) off += s_wcnt[w];
            n += s_wcnt[w];
        }
        if (keep) s_tok[off + __popc(m & ((1u << lane) - 1u))] = packed;
        __syncthreads();
        // this half-warp's tokens of the round: t = par, par + 4, ... (ascending token index)
        for (int t0 = par; t0 < n; t0 += 4 * INS_UNROLL) {
            uint32_t e[INS_UNROLL];
            uint4 x[INS_UNROLL];
#pragma unroll
            for (int q = 0; q < INS_UNROLL; ++q) {
                const int t = t0 + 4 * q;
                e[q] = (t < n) ? s_tok[t] : 0xFFFFFFFFu;
                if (t < n) x[q] = src[(size_t)(e[q] & 0x7FFFFFFFu) * (KVR_D / 8)];
            }
#pragma unroll
            for (int d = 0; d < 8; ++d) blk[d] = 0.f;
#pragma unroll
            for (int q = 0; q < INS_UNROLL; ++q)
                if (t0 + 4 * q < n) add(x[q], e[q]);
            fold();
        }
        __syncthreads();
    }
    // (tokens 0 mod 4 + tokens 1 mod 4) + (tokens 2 mod 4 + tokens 3 mod 4), in that order
    float mine[8];
#pragma unroll
    for (int d = 0; d < 8; ++d) {
        mine[d] = s[d] + cc[d];
        mine[d] += __shfl_down_sync(0xFFFFFFFFu, mine[d], 16);                  // (meaningful in the lower half-warp)
    }
    const bool upper = (warp >> 1) != 0;
    if (upper && lane < 16) {
        s_part[kv][2 * l16] = make_float4(mine[0], mine[1], mine[2], mine[3]);
        s_part[kv][2 * l16 + 1] = make_float4(mine[4], mine[5], mine[6], mine[7]);
    }
    __syncthreads();
    if (!upper && lane < 16) {
        const float4 o0 = s_part[kv][2 * l16], o1 = s_part[kv][2 * l16 + 1];
        float* cell = cells_all + ((((size_t)inst * 2 + kv) * r + i) * b + c) * KVR_D + 8 * l16;
        *reinterpret_cast<float4*>(cell) = make_float4(mine[0] + o0.x, mine[1] + o0.y, mine[2] + o0.z, mine[3] + o0.w);
        *reinterpret_cast<float4*>(cell + 4) = make_float4(mine[4] + o1.x, mine[5] + o1.y, mine[6] + o1.z, mine[7] + o1.w);
    }
}

// One warp per compressed token, 4 channels per lane.
__global__ void reconstruct_kernel(const float* __restrict__ cells_all, const int32_t* __restrict__ cmp_all,
                                   const int32_t* __restrict__ tok_h, const int8_t* __restrict__ tok_g,
                                   int max_ctx, int b, int a, int inst0, int n_tbl, int mean, float* __restrict__ Kt,
                                   float* __restrict__ Vt) {
    const int u = blockIdx.y, inst = inst0 + u;
    const int tb = n_tbl > 1 ? inst % n_tbl : 0;
    tok_h += (size_t)tb * KVR_R * max_ctx;
    tok_g += (size_t)tb * KVR_R * max_ctx;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (t >= a) return;
    const int J = cmp_all[(size_t)inst * max_ctx + t];
    const float* ck = cells_all + (size_t)inst * 2 * KVR_R * b * KVR_D;
    const float* cv = ck + (size_t)KVR_R * b * KVR_D;
    float4 k[KVR_R], v[KVR_R];
#pragma unroll
    for (int i = 0; i < KVR_R; ++i) {
        const int h = tok_h[(size_t)i * max_ctx + J];
        const float g = (float)tok_g[(size_t)i * max_ctx + J];
        k[i] = *reinterpret_cast<const float4*>(ck + ((size_t)i * b + h) * KVR_D + 4 * lane);
        float4 x = *reinterpret_cast<const float4*>(cv + ((size_t)i * b + h) * KVR_D + 4 * lane);
        v[i] = make_float4(g * x.x, g * x.y, g * x.z, g * x.w);
    }
    float4 ko = make_float4(kvr_comb3(k[0].x, k[1].x, k[2].x, mean), kvr_comb3(k[0].y, k[1].y, k[2].y, mean),
                            kvr_comb3(k[0].z, k[1].z, k[2].z, mean), kvr_comb3(k[0].w, k[1].w, k[2].w, mean));
    float4 vo = make_float4(kvr_comb3(v[0].x, v[1].x, v[2].x, mean), kvr_comb3(v[0].y, v[1].y, v[2].y, mean),
                            kvr_comb3(v[0].z, v[1].z, v[2].z, mean), kvr_comb3(v[0].w, v[1].w, v[2].w, mean));
    const size_t o = ((size_t)u * a + t) * KVR_D + 4 * lane;
    if (Kt) *reinterpret_cast<float4*>(Kt + o) = ko;
    if (Vt) *reinterpret_cast<float4*>(Vt + o) = vo;
}

}  // namespace

cudaError_t kvr_launch_insert(kvr_sketch* sk, int inst0, int n_inst, int N, const void* K, const void* V,
                              cudaStream_t st) {
    dim3 g(sk->d.b, sk->d.r, n_inst);
    // (follows the copy of the retained rows, or the selection, of the same compress on `st`)
    cudaError_t e;
    if (sk->d.kv_dtype == KVR_F16)
        e = kvr_launch_after(insert_kernel<__half>, g, dim3(INS_THREADS), 0, st, true, (const int32_t*)sk->full_off,
                             (const int32_t*)sk->full_list, (const int8_t*)sk->tok_g, (const uint32_t*)sk->bitmap, sk->bitmap_words,
                             (const uint4*)K, (const uint4*)V, N, sk->d.max_context, sk->d.b, inst0, sk->n_tbl, sk->d.r, sk->cells);
    else
        e = kvr_launch_after(insert_kernel<__nv_bfloat16>, g, dim3(INS_THREADS), 0, st, true, (const int32_t*)sk->full_off,
                             (const int32_t*)sk->full_list, (const int8_t*)sk->tok_g, (const uint32_t*)sk->bitmap, sk->bitmap_words,
                             (const uint4*)K, (const uint4*)V, N, sk->d.max_context, sk->d.b, inst0, sk->n_tbl, sk->d.r, sk->cells);
    sk->launches += 1;
    return e;
}

cudaError_t kvr_launch_reconstruct(const kvr_sketch* sk, int inst0, int n_inst, int a, float* Kt, float* Vt,
                                   cudaStream_t st) {
    if (a <= 0 || n_inst <= 0) return cudaSuccess;
    dim3 g((a + 7) / 8, n_inst);
    reconstruct_kernel<<<g, 256, 0, st>>>(sk->cells, sk->cmp_idx, sk->tok_h, sk->tok_g, sk->d.max_context,
                                          sk->d.b, a, inst0, sk->n_tbl, sk->combine, Kt, Vt);
    const_cast<kvr_sketch*>(sk)->launches += 1;
    return cudaGetLastError();
}
