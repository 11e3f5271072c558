// Decode attention over the mixed cache: Algorithm 4 (Revive) fused with the attention of the
// Calculation Phase, p = Softmax(q K^T / sqrt(d_k)), out = p V, over all N tokens of a layer.
// Retained tokens contribute their exact rows; a compressed token J contributes
//     K~_J[d] = median_i cellK[i][h_i(J)][d],   V~_J[d] = median_i g_i(J) cellV[i][h_i(J)][d]
// (Algorithm 2) computed in registers -- the rebuilt [N, d] cache is never written anywhere.
//
// General kernel (any b): split-KV.  CTA (s, u) handles slice s of the retained rows and of the
// compressed-token list of head-instance u, keeps one online-softmax state per half-warp (16 lanes
// x 8 channels), merges the states in shared memory and writes one partial (max, sum, o[G][128]).
// The CTA that arrives last at a per-instance ticket merges all partials into `out`: no waiting.
// The compressed list is ordered by row-0 cell, so that cell stays in registers while its tokens
// are processed; the other two cells are fetched from global memory (L1/L2).
#include <mutex>

#include "kvr_internal.h"

namespace {

constexpr int DEC_THREADS = 256;
constexpr int DEC_PART = KVR_D + 2;   // o[128], max, sum

struct DecodeParams {
    const uint4* q;        // [n_inst][G][16]   (16-bit x 8 per uint4)
    const uint4* Kr;       // [n_inst][R][16]
    const uint4* Vr;
    const float* cells;    // handle base: [inst][2][r][b][D]
    const uint32_t* dlist; // handle base: [inst][max_ctx]
    const int32_t* doff;   // handle base: [inst][b+1]
    float* part;           // [n_inst][S][G][DEC_PART]
    uint32_t* tickets;     // arrival counters; head-instance u of the call uses slot ticket0 + u
    int ticket0;
    float* out;            // [n_inst][G][D]
    float* ml;             // handle base: [inst][G][2] maximum (log2 units) and sum of the softmax
    int inst0, R, a, b, max_ctx, n_splits;
    int mean;              // combine of the three cells: 0 median, 1 mean
    float scale_log2e;
};

template <typename T>
__device__ __forceinline__ void unpack8(const uint4& x, float (&f)[8]) {
    float2 a = KvrType<T>::to_f2(x.x), b = KvrType<T>::to_f2(x.y), c = KvrType<T>::to_f2(x.z),
           d = KvrType<T>::to_f2(x.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

__device__ __forceinline__ void load8(const float* p, float (&f)[8]) {
    float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
}

__device__ __forceinline__ float safe_exp2_diff(float m, float M) {
    return (m == -INFINITY) ? 0.f : exp2f(m - M);
}

template <typename T, int G>
__global__ void __launch_bounds__(DEC_THREADS)
decode_split_kernel(const DecodeParams p) {
    __shared__ float s_o[DEC_THREADS / 32][G][KVR_D];
    __shared__ float s_m[DEC_THREADS / 32][G], s_l[DEC_THREADS / 32][G];
    __shared__ int s_last;

    const int u = blockIdx.y, inst = p.inst0 + u, sp = blockIdx.x, S = p.n_splits;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, hw = tid >> 4, l16 = tid & 15;

    float qf[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        unpack8<T>(p.q[((size_t)u * G + g) * 16 + l16], qf[g]);
#pragma unroll
        for (int e = 0; e < 8; ++e) qf[g][e] *= p.scale_log2e;
    }
    float m[G], l[G], o[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
        m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) o[g][e] = 0.f;
    }

    auto accumulate = [&](bool valid, const float (&kf)[8], const float (&vf)[8], float vscale) {
        float s[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            float acc = 0.f;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc = fmaf(qf[g][e], kf[e], acc);
            s[g] = acc;
        }
#pragma unroll
        for (int off = 8; off > 0; off >>= 1)
#pragma unroll
            for (int g = 0; g < G; ++g) s[g] += __shfl_xor_sync(0xFFFFFFFFu, s[g], off);
        if (valid) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                if (s[g] > m[g]) {
                    const float c = exp2f(m[g] - s[g]);
                    l[g] *= c;
#pragma unroll
                    for (int e = 0; e < 8; ++e) o[g][e] *= c;
                    m[g] = s[g];
                }
                const float pr = exp2f(s[g] - m[g]);
                l[g] += pr;
                const float pv = pr * vscale;
#pragma unroll
                for (int e = 0; e < 8; ++e) o[g][e] = fmaf(pv, vf[e], o[g][e]);
            }
        }
    };

    // ---- retained tokens: exact rows -------------------------------------------------------
    {
        const int r_begin = (int)((long long)p.R * sp / S), r_end = (int)((long long)p.R * (sp + 1) / S);
        const uint4* Kr = p.Kr + (size_t)u * p.R * 16 + l16;
        const uint4* Vr = p.Vr + (size_t)u * p.R * 16 + l16;
        for (int base = r_begin; base < r_end; base += DEC_THREADS / 16) {
            const int t = base + hw;
            const bool valid = t < r_end;
            const int tt = valid ? t : r_begin;
            float kf[8], vf[8];
            unpack8<T>(Kr[(size_t)tt * 16], kf);
            unpack8<T>(Vr[(size_t)tt * 16], vf);
            accumulate(valid, kf, vf, 1.f);
        }
    }

    // ---- compressed tokens: median of three cells -------------------------------------------
    if (p.a > 0) {
        const int a_begin = (int)((long long)p.a * sp / S), a_end = (int)((long long)p.a * (sp + 1) / S);
        if (a_end > a_begin) {
            const int b = p.b;
            const int32_t* doff = p.doff + (size_t)inst * (b + 1);
            const uint32_t* dlist = p.dlist + (size_t)inst * p.max_ctx;
            const float* cK = p.cells + (size_t)inst * 2 * KVR_R * b * KVR_D + l16 * 8;
            const float* cV = cK + (size_t)KVR_R * b * KVR_D;
            // largest cell c with doff[c] <= a_begin
            int lo = 0, hi = b;
            while (hi - lo > 1) {
                int mid = (lo + hi) >> 1;
                if (doff[mid] <= a_begin) lo = mid; else hi = mid;
            }
            for (int c = lo; c < b; ++c) {
                const int d0 = doff[c], d1 = doff[c + 1];
                if (d0 >= a_end) break;
                const int p0 = max(d0, a_begin), p1 = min(d1, a_end);
                if (p1 <= p0) continue;
                float k0[8], v0[8];
                load8(cK + (size_t)c * KVR_D, k0);
                load8(cV + (size_t)c * KVR_D, v0);
                for (int base = p0; base < p1; base += DEC_THREADS / 16) {
                    const int pos = base + hw;
                    const bool valid = pos < p1;
                    const uint32_t e = valid ? dlist[pos] : 0u;
                    const uint32_t h1 = e & KVR_PACK_H_MASK, h2 = (e >> KVR_PACK_H2_SHIFT) & KVR_PACK_H_MASK;
                    const uint32_t sg = e >> KVR_PACK_SIGN_SHIFT;
                    float k1[8], k2[8], kf[8];
                    load8(cK + ((size_t)b + h1) * KVR_D, k1);
                    load8(cK + ((size_t)2 * b + h2) * KVR_D, k2);
#pragma unroll
                    for (int x = 0; x < 8; ++x) kf[x] = kvr_comb3(k0[x], k1[x], k2[x], p.mean);
                    // median and mean are odd: f(g0 a, g1 b, g2 c) = g0 f(a, g0 g1 b, g0 g2 c)
                    const float g0 = (sg & 1u) ? -1.f : 1.f;
                    const float g01 = ((sg ^ (sg >> 1)) & 1u) ? -1.f : 1.f;
                    const float g02 = ((sg ^ (sg >> 2)) & 1u) ? -1.f : 1.f;
                    float v1[8], v2[8], vf[8];
                    load8(cV + ((size_t)b + h1) * KVR_D, v1);
                    load8(cV + ((size_t)2 * b + h2) * KVR_D, v2);
#pragma unroll
                    for (int x = 0; x < 8; ++x) vf[x] = kvr_comb3(v0[x], g01 * v1[x], g02 * v2[x], p.mean);
                    accumulate(valid, kf, vf, g0);
                }
            }
        }
    }

    // ---- merge the two half-warps of each warp, then the 8 warps -------------------------------
#pragma unroll
    for (int g = 0; g < G; ++g) {
        const float mo = __shfl_xor_sync(0xFFFFFFFFu, m[g], 16);
        const float lo_ = __shfl_xor_sync(0xFFFFFFFFu, l[g], 16);
        const float M = fmaxf(m[g], mo);
        const float cs = safe_exp2_diff(m[g], M), co = safe_exp2_diff(mo, M);
        l[g] = l[g] * cs + lo_ * co;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float oo = __shfl_xor_sync(0xFFFFFFFFu, o[g][e], 16);
            o[g][e] = o[g][e] * cs + oo * co;
        }
        m[g] = M;
        if (lane < 16) {
#pragma unroll
            for (int e = 0; e < 8; ++e) s_o[warp][g][l16 * 8 + e] = o[g][e];
            if (lane == 0) { s_m[warp][g] = m[g]; s_l[warp][g] = l[g]; }
        }
    }
    __syncthreads();
    float* part = p.part + ((size_t)u * S + sp) * G * DEC_PART;
    for (int idx = tid; idx < G * KVR_D; idx += DEC_THREADS) {
        const int g = idx >> 7, d = idx & (KVR_D - 1);
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < DEC_THREADS / 32; ++w) M = fmaxf(M, s_m[w][g]);
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int w = 0; w < DEC_THREADS / 32; ++w) {
            const float f = safe_exp2_diff(s_m[w][g], M);
            L += s_l[w][g] * f;
            O += s_o[w][g][d] * f;
        }
        part[g * DEC_PART + d] = O;
        if (d == 0) { part[g * DEC_PART + KVR_D] = M; part[g * DEC_PART + KVR_D + 1] = L; }
    }

    // ---- last CTA of this head-instance merges the splits ------------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned t = atomicAdd(&p.tickets[p.ticket0 + u], 1u);
        s_last = (t == (unsigned)(S - 1));
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    const float* pu = p.part + (size_t)u * S * G * DEC_PART;
    for (int idx = tid; idx < G * KVR_D; idx += DEC_THREADS) {
        const int g = idx >> 7, d = idx & (KVR_D - 1);
        float M = -INFINITY;
        for (int s = 0; s < S; ++s) M = fmaxf(M, __ldcg(pu + ((size_t)s * G + g) * DEC_PART + KVR_D));
        float L = 0.f, O = 0.f;
        for (int s = 0; s < S; ++s) {
            const float* ps = pu + ((size_t)s * G + g) * DEC_PART;
            const float f = safe_exp2_diff(__ldcg(ps + KVR_D), M);
            L += __ldcg(ps + KVR_D + 1) * f;
            O += __ldcg(ps + d) * f;
        }
        p.out[((size_t)u * G + g) * KVR_D + d] = O / L;
        if (d == 0) { p.ml[((size_t)inst * G + g) * 2] = M; p.ml[((size_t)inst * G + g) * 2 + 1] = L; }
    }
    if (tid == 0) p.tickets[p.ticket0 + u] = 0u;
}

template <typename T>
cudaError_t launch_G(const DecodeParams& p, int G, dim3 grid, cudaStream_t st) {
    switch (G) {
        case 1: decode_split_kernel<T, 1><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 2: decode_split_kernel<T, 2><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 4: decode_split_kernel<T, 4><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 8: decode_split_kernel<T, 8><<<grid, DEC_THREADS, 0, st>>>(p); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

}  // namespace

size_t kvr_decode_ws_bytes(int n_inst, int n_splits, int G) {
    return sizeof(float) * (size_t)n_inst * n_splits * G * DEC_PART;
}

// Enough CTAs to fill the machine about three times over, at least ~128 tokens per split.
int kvr_decode_pick_splits(const kvr_sketch* sk, int n_inst, int N, int R) {
    (void)R;
    int want = (3 * sk->n_sm + n_inst - 1) / n_inst;
    int cap = (N + 127) / 128;
    int s = want < cap ? want : cap;
    if (s < 1) s = 1;
    if (s > 128) s = 128;
    return s;
}

cudaError_t kvr_launch_decode(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                              const void* Kr, const void* Vr, float scale, float* out, int n_splits,
                              cudaStream_t st) {
    DecodeParams p;
    p.q = (const uint4*)q;
    p.Kr = (const uint4*)Kr;
    p.Vr = (const uint4*)Vr;
    p.cells = sk->cells;
    p.dlist = sk->dlist;
    p.doff = sk->doff;
    p.part = (float*)sk->ws_decode;
    p.tickets = sk->tickets;
    p.ticket0 = inst0;
    p.out = out;
    p.ml = sk->ml;
    p.mean = sk->combine;
    p.inst0 = inst0;
    p.R = rows;
    p.a = N - R;
    p.b = sk->d.b;
    p.max_ctx = sk->d.max_context;
    p.n_splits = n_splits;
    p.scale_log2e = scale * 1.4426950408889634f;
    dim3 grid(n_splits, n_inst);
    sk->launches += 1;
    if (sk->d.kv_dtype == KVR_F16) return launch_G<__half>(p, sk->G, grid, st);
    return launch_G<__nv_bfloat16>(p, sk->G, grid, st);
}

// ================================================================================================
// Allocation-free decode call.
//
// Same kernel as kvr_launch_decode, but the split partials and the arrival tickets live in one
// fixed array in device global memory that is part of this library's image, so the call never
// asks the CUDA allocator for anything.  It is meant for hosts that cannot allocate at decode
// time: a serving process that has already handed all free device memory to its own pool (a
// cudaMalloc there fails, or steals from the pool's head-room), or a decode loop that must not
// take the device-wide synchronisation that cudaMalloc / cudaFree imply.
// ================================================================================================
#define KVR_STATIC_TICKET_SLOTS 4096u
static __device__ __align__(256) unsigned char kvr_static_scratch[KVR_STATIC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
unsigned char* g_static_scratch_ptr[kMaxDevices];   // device address of kvr_static_scratch, per device

// The array's name is only a host-side stand-in; the address a kernel can use has to be asked for,
// once per device, with that device current.
std::mutex g_static_scratch_mutex;                   // two handles on two host threads may make their first call together
cudaError_t static_scratch_address(int device, unsigned char** out) {
    if (device < 0 || device >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ptr[device]) {
        unsigned char* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void**)&ptr, kvr_static_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_static_scratch_ptr[device] = ptr;
    }
    *out = g_static_scratch_ptr[device];
    return cudaSuccess;
}
}  // namespace

extern "C" kvr_status_t kvr_decode_attention_static(kvr_sketch_t* sk, int32_t layer, const void* q, const void* Kr,
                                                    const void* Vr, const int32_t* ret_idx, int32_t n_retained,
                                                    float softmax_scale, float* out, void* cuda_stream) {
    (void)ret_idx;
    if (!sk || !q || !out) return KVR_ERR_INVALID_ARG;
    auto misaligned = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
    if (misaligned(q) || misaligned(Kr) || misaligned(Vr) || misaligned(out)) return KVR_ERR_INVALID_ARG;
    if (!(softmax_scale >= 0.f) || isinf(softmax_scale)) return KVR_ERR_INVALID_ARG;
    if (sk->d.r != KVR_R) return KVR_ERR_UNSUPPORTED;          // the split kernel behind this call is written for r = 3
    int inst0, n_inst, layer0, n_layers;
    if (layer == KVR_ALL_LAYERS) { inst0 = 0; n_inst = sk->n_inst; layer0 = 0; n_layers = sk->d.n_layers; }
    else if (layer >= 0 && layer < sk->d.n_layers) { inst0 = layer * sk->BH; n_inst = sk->BH; layer0 = layer; n_layers = 1; }
    else return KVR_ERR_SHAPE;
    const int N = sk->layer_N[layer0], R = sk->layer_R[layer0];
    if (N < 0) return KVR_ERR_STATE;
    for (int l = layer0; l < layer0 + n_layers; ++l) {
        if (sk->layer_N[l] < 0) return KVR_ERR_STATE;
        if (sk->layer_N[l] != N || sk->layer_R[l] != R) return KVR_ERR_SHAPE;
    }
    if (n_retained < R) return KVR_ERR_SHAPE;          // rows beyond R: tokens appended after the compress
    if (n_retained > 0 && (!Kr || !Vr)) return KVR_ERR_INVALID_ARG;

    // scratch layout: [0, 16 KiB) one ticket per head-instance of the call, then the split partials
    const int S = kvr_decode_pick_splits(sk, n_inst, N, R);
    const size_t ticket_bytes = sizeof(uint32_t) * KVR_STATIC_TICKET_SLOTS;
    if ((unsigned)n_inst > KVR_STATIC_TICKET_SLOTS ||
        kvr_decode_ws_bytes(n_inst, S, sk->G) > (size_t)KVR_STATIC_SCRATCH_BYTES - ticket_bytes)
        return KVR_ERR_LIMIT;

    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) return KVR_ERR_CUDA;
    if (prev != sk->device && cudaSetDevice(sk->device) != cudaSuccess) return KVR_ERR_CUDA;
    kvr_status_t rc = KVR_OK;
    unsigned char* scratch = nullptr;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (static_scratch_address(sk->device, &scratch) != cudaSuccess) rc = KVR_ERR_CUDA;
    // The array keeps whatever the previous call left: the tickets must start at zero.
    if (rc == KVR_OK && cudaMemsetAsync(scratch, 0, sizeof(uint32_t) * n_inst, st) != cudaSuccess) rc = KVR_ERR_CUDA;
    if (rc == KVR_OK) {
        if (softmax_scale == 0.f) softmax_scale = 1.0f / sqrtf((float)sk->d.head_dim);
        DecodeParams p;
        p.q = (const uint4*)q;
        p.Kr = (const uint4*)Kr;
        p.Vr = (const uint4*)Vr;
        p.cells = sk->cells;
        p.dlist = sk->dlist;
        p.doff = sk->doff;
        p.part = reinterpret_cast<float*>(scratch + ticket_bytes);
        p.tickets = reinterpret_cast<uint32_t*>(scratch);        // slot 0 belongs to the call's first head-instance
        p.ticket0 = 0;
        p.out = out;
        p.ml = sk->ml;
        p.mean = sk->combine;
        p.inst0 = inst0;
        p.R = n_retained;
        p.a = N - R;
        p.b = sk->d.b;
        p.max_ctx = sk->d.max_context;
        p.n_splits = S;
        p.scale_log2e = softmax_scale * 1.4426950408889634f;
        dim3 grid(S, n_inst);
        sk->launches += 1;
        cudaError_t e = (sk->d.kv_dtype == KVR_F16) ? launch_G<__half>(p, sk->G, grid, st)
                                                    : launch_G<__nv_bfloat16>(p, sk->G, grid, st);
        if (e != cudaSuccess) rc = KVR_ERR_CUDA;
        else sk->last_decode_kernel = KVR_DECODE_SPLIT;
    }
    if (prev != sk->device) cudaSetDevice(prev);
    return rc;
}
