// Decode attention and reconstruction for sketches with r = 1 or r = 5 rows (the Vague Sketch section
// has "r distinct hash functions"; the Parameter Settings appendix fixes r = 3 as the chosen value, which
// the fast kernels are written for).  Algorithm 2's element-wise median over r collected numbers is
// written out for each r: the number itself (r = 1: a direct look-up), the middle of three, the middle
// of five; Algorithm 4 + Softmax(q K^T / sqrt(d_k)) V as in the other decode kernels.
//
// Plain and general rather than fast: a warp takes one token at a time (4 channels per lane), looks
// the token's r cells up through the hash tables and reads them through L1/L2; split-KV over the
// retained rows followed by the compressed tokens; the CTA that arrives last merges the partials.
#include "kvr_decode_common.cuh"

namespace {
using namespace kvr_dec;

constexpr int GEN_THREADS = 256, GEN_WARPS = GEN_THREADS / 32;
constexpr unsigned FULL = 0xFFFFFFFFu;

// middle of r numbers (r odd), or their mean
template <int R>
__device__ __forceinline__ float combine(const float (&x)[R], int mean) {
    if (mean) {
        float s = x[0];
#pragma unroll
        for (int i = 1; i < R; ++i) s += x[i];
        return s * (1.0f / R);
    }
    if constexpr (R == 1) return x[0];
    else if constexpr (R == 3) return kvr_med3(x[0], x[1], x[2]);
    else {
        // of five: drop the smallest and the largest of the first four, then the middle of three
        const float f = fmaxf(fminf(x[0], x[1]), fminf(x[2], x[3]));
        const float g = fminf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        return kvr_med3(x[4], f, g);
    }
}

// K~ / V~ of token J on this lane's 4 channels
template <int R>
__device__ __forceinline__ void query_token(const float* __restrict__ ck, const float* __restrict__ cv,
                                            const int32_t* __restrict__ tok_h, const int8_t* __restrict__ tok_g,
                                            int max_ctx, int b, int J, int lane, int mean, float4* k, float4* v) {
    float kx[R], ky[R], kz[R], kw[R], vx[R], vy[R], vz[R], vw[R];
#pragma unroll
    for (int i = 0; i < R; ++i) {
        const int h = tok_h[(size_t)i * max_ctx + J];
        const float g = (float)tok_g[(size_t)i * max_ctx + J];
        const float4 a = *reinterpret_cast<const float4*>(ck + ((size_t)i * b + h) * KVR_D + 4 * lane);
        kx[i] = a.x; ky[i] = a.y; kz[i] = a.z; kw[i] = a.w;
        if (v) {
            const float4 c = *reinterpret_cast<const float4*>(cv + ((size_t)i * b + h) * KVR_D + 4 * lane);
            vx[i] = g * c.x; vy[i] = g * c.y; vz[i] = g * c.z; vw[i] = g * c.w;
        }
    }
    *k = make_float4(combine<R>(kx, mean), combine<R>(ky, mean), combine<R>(kz, mean), combine<R>(kw, mean));
    if (v) *v = make_float4(combine<R>(vx, mean), combine<R>(vy, mean), combine<R>(vz, mean), combine<R>(vw, mean));
}

struct GenParams {
    const uint2* q;        // [n_inst][G][32]   4 channels (8 bytes) per lane
    const uint2* Kr;       // [n_inst][rows][32]
    const uint2* Vr;
    const float* cells;    // handle base: [inst][2][r][b][128]
    const int32_t* cmp;    // handle base: [inst][max_ctx]
    const int32_t* tok_h;  // [n_tbl][r][max_ctx]
    const int8_t* tok_g;
    float* part;           // [n_inst][splits][G][PART]
    uint32_t* tickets;     // handle base: [inst]
    float* out;            // [n_inst][G][128]
    float* ml;             // handle base: [inst][G][2]
    int inst0, rows, a, b, max_ctx, n_tbl, mean;
    float scale_log2e;
};

template <typename T, int G, int R>
__global__ void __launch_bounds__(GEN_THREADS)
decode_generic_kernel(const GenParams p) {
    __shared__ float s_o[GEN_WARPS][G][KVR_D];
    __shared__ float s_m[GEN_WARPS][G], s_l[GEN_WARPS][G];
    __shared__ int s_flag;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.y, inst = p.inst0 + u, sp = blockIdx.x, S = gridDim.x;
    const int tb = p.n_tbl > 1 ? inst % p.n_tbl : 0;
    const int32_t* tok_h = p.tok_h + (size_t)tb * R * p.max_ctx;
    const int8_t* tok_g = p.tok_g + (size_t)tb * R * p.max_ctx;
    const float* ck = p.cells + (size_t)inst * 2 * R * p.b * KVR_D;
    const float* cv = ck + (size_t)R * p.b * KVR_D;
    const int32_t* cmp = p.cmp + (size_t)inst * p.max_ctx;

    float4 q[G];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const uint2 x = p.q[((size_t)u * G + g) * 32 + lane];
        const float2 lo = KvrType<T>::to_f2(x.x), hi = KvrType<T>::to_f2(x.y);
        q[g] = make_float4(lo.x * p.scale_log2e, lo.y * p.scale_log2e, hi.x * p.scale_log2e, hi.y * p.scale_log2e);
    }
    float m[G], l[G];
    float4 o[G];
#pragma unroll
    for (int g = 0; g < G; ++g) { m[g] = M_EMPTY; l[g] = 0.f; o[g] = make_float4(0.f, 0.f, 0.f, 0.f); }

    const int total = p.rows + p.a;
    const int per = (total + S - 1) / S;
    const int t0 = min(sp * per, total), t1 = min(t0 + per, total);
    for (int t = t0 + warp; t < t1; t += GEN_WARPS) {             // (uniform per warp)
        float4 k, v;
        if (t < p.rows) {                                          // Algorithm 4: an exact row
            const uint2 kx = p.Kr[((size_t)u * p.rows + t) * 32 + lane], vx = p.Vr[((size_t)u * p.rows + t) * 32 + lane];
            const float2 a = KvrType<T>::to_f2(kx.x), c = KvrType<T>::to_f2(kx.y);
            const float2 d = KvrType<T>::to_f2(vx.x), e = KvrType<T>::to_f2(vx.y);
            k = make_float4(a.x, a.y, c.x, c.y);
            v = make_float4(d.x, d.y, e.x, e.y);
        } else {                                                   // Algorithm 4: a vague token, Algorithm 2
            query_token<R>(ck, cv, tok_h, tok_g, p.max_ctx, p.b, cmp[t - p.rows], lane, p.mean, &k, &v);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float s = q[g].x * k.x + q[g].y * k.y + q[g].z * k.z + q[g].w * k.w;
#pragma unroll
            for (int x = 16; x >= 1; x >>= 1) s += __shfl_xor_sync(FULL, s, x);
            const float mn = fmaxf(m[g], s);
            const float c = ex2(m[g] - mn), pr = ex2(s - mn);
            l[g] = l[g] * c + pr;
            o[g] = make_float4(o[g].x * c + pr * v.x, o[g].y * c + pr * v.y, o[g].z * c + pr * v.z, o[g].w * c + pr * v.w);
            m[g] = mn;
        }
    }
    // ---- the CTA's partial: warps folded in warp order
#pragma unroll
    for (int g = 0; g < G; ++g) {
        *reinterpret_cast<float4*>(&s_o[warp][g][4 * lane]) = o[g];
        if (lane == 0) { s_m[warp][g] = m[g]; s_l[warp][g] = l[g]; }
    }
    __syncthreads();
    float* part = p.part + ((size_t)u * S + sp) * G * PART;
    for (int idx = tid; idx < G * KVR_D; idx += GEN_THREADS) {
        const int g = idx >> 7, d = idx & (KVR_D - 1);
        float M = M_EMPTY;
#pragma unroll
        for (int w = 0; w < GEN_WARPS; ++w) M = fmaxf(M, s_m[w][g]);
        float Ls = 0.f, Os = 0.f;
#pragma unroll
        for (int w = 0; w < GEN_WARPS; ++w) {
            const float f = ex2(s_m[w][g] - M);
            Ls += s_l[w][g] * f;
            Os += s_o[w][g][d] * f;
        }
        part[g * PART + d] = Os;
        if (d == 0) { part[g * PART + KVR_D] = M; part[g * PART + KVR_D + 1] = Ls; }
    }
    finish_instance<G, GEN_THREADS>(p.part + (size_t)u * S * G * PART, S, &p.tickets[inst], p.out + (size_t)u * G * KVR_D,
                                    p.ml + (size_t)inst * G * 2, &s_flag);
}

// One warp per compressed token, 4 channels per lane.
template <int R>
__global__ void reconstruct_generic_kernel(const float* __restrict__ cells_all, const int32_t* __restrict__ cmp_all,
                                           const int32_t* __restrict__ tok_h, const int8_t* __restrict__ tok_g,
                                           int max_ctx, int b, int a, int inst0, int n_tbl, int mean,
                                           float* __restrict__ Kt, float* __restrict__ Vt) {
    const int u = blockIdx.y, inst = inst0 + u;
    const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (t >= a) return;
    const int tb = n_tbl > 1 ? inst % n_tbl : 0;
    const float* ck = cells_all + (size_t)inst * 2 * R * b * KVR_D;
    float4 k, v;
    query_token<R>(ck, ck + (size_t)R * b * KVR_D, tok_h + (size_t)tb * R * max_ctx, tok_g + (size_t)tb * R * max_ctx, max_ctx, b,
                   cmp_all[(size_t)inst * max_ctx + t], lane, mean, &k, &v);
    const size_t o = ((size_t)u * a + t) * KVR_D + 4 * lane;
    if (Kt) *reinterpret_cast<float4*>(Kt + o) = k;
    if (Vt) *reinterpret_cast<float4*>(Vt + o) = v;
}

template <typename T, int R>
cudaError_t launch_R(const GenParams& p, int G, dim3 grid, cudaStream_t st) {
    switch (G) {
        case 1: decode_generic_kernel<T, 1, R><<<grid, GEN_THREADS, 0, st>>>(p); break;
        case 2: decode_generic_kernel<T, 2, R><<<grid, GEN_THREADS, 0, st>>>(p); break;
        case 4: decode_generic_kernel<T, 4, R><<<grid, GEN_THREADS, 0, st>>>(p); break;
        case 8: decode_generic_kernel<T, 8, R><<<grid, GEN_THREADS, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

// Decode attention of a handle with r = 1 or r = 5 rows; part: n_inst x n_splits x G x PART floats.
cudaError_t kvr_launch_decode_generic(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                                      const void* Kr, const void* Vr, float scale, float* out, int n_splits,
                                      cudaStream_t st) {
    GenParams p;
    p.q = (const uint2*)q;
    p.Kr = (const uint2*)Kr;
    p.Vr = (const uint2*)Vr;
    p.cells = sk->cells;
    p.cmp = sk->cmp_idx;
    p.tok_h = sk->tok_h;
    p.tok_g = sk->tok_g;
    p.part = (float*)sk->ws_decode;
    p.tickets = sk->tickets;
    p.out = out;
    p.ml = sk->ml;
    p.inst0 = inst0;
    p.rows = rows;
    p.a = N - R;
    p.b = sk->d.b;
    p.max_ctx = sk->d.max_context;
    p.n_tbl = sk->n_tbl;
    p.mean = sk->combine;
    p.scale_log2e = scale * 1.4426950408889634f;
    const dim3 grid(n_splits, n_inst);
    sk->launches += 1;
    const bool f16 = sk->d.kv_dtype == KVR_F16;
    if (sk->d.r == 1) return f16 ? launch_R<__half, 1>(p, sk->G, grid, st) : launch_R<__nv_bfloat16, 1>(p, sk->G, grid, st);
    if (sk->d.r == 5) return f16 ? launch_R<__half, 5>(p, sk->G, grid, st) : launch_R<__nv_bfloat16, 5>(p, sk->G, grid, st);
    return cudaErrorInvalidValue;
}

cudaError_t kvr_launch_reconstruct_generic(const kvr_sketch* sk, int inst0, int n_inst, int a, float* Kt, float* Vt,
                                           cudaStream_t st) {
    if (a <= 0 || n_inst <= 0) return cudaSuccess;
    const dim3 g((a + 7) / 8, n_inst);
    if (sk->d.r == 1)
        reconstruct_generic_kernel<1><<<g, 256, 0, st>>>(sk->cells, sk->cmp_idx, sk->tok_h, sk->tok_g, sk->d.max_context, sk->d.b,
                                                         a, inst0, sk->n_tbl, sk->combine, Kt, Vt);
    else if (sk->d.r == 5)
        reconstruct_generic_kernel<5><<<g, 256, 0, st>>>(sk->cells, sk->cmp_idx, sk->tok_h, sk->tok_g, sk->d.max_context, sk->d.b,
                                                         a, inst0, sk->n_tbl, sk->combine, Kt, Vt);
    else
        return cudaErrorInvalidValue;
    const_cast<kvr_sketch*>(sk)->launches += 1;
    return cudaGetLastError();
}
