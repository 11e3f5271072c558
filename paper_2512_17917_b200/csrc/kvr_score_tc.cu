// Importance scoring on the fifth-generation tensor cores (tcgen05 + tensor memory + TMA).
//
// Same two passes as kvr_score.cu (row maximum / row sum per chunk of keys, then the column sums of
// the normalised probabilities; the per-chunk statistics are folded by pass 2 itself), but the
// logits tile S = Qobs . K^T [128 x 128] is produced by tcgen05.mma from operands that TMA places in
// shared memory (128-byte swizzle, K-major), accumulates in tensor memory, and is read back one row
// per thread (tcgen05.ld 32x32b): the softmax statistics of a row are thread-local, and the column
// sums are a transposing shuffle tree over the 32 rows of a warp.
//
// Warp roles in a CTA of 320 threads:
//   warp 0      one lane issues the TMA loads (Q once per m-tile, a ring of two key tiles)
//   warp 1      allocates 256 tensor-memory columns (two accumulator buffers); one lane issues the MMAs
//   warps 2..9  epilogue: warp w reads the 32 rows of lane quarter w % 4, half of the 128 columns each
// Every wait on an mbarrier is bounded in time: a wait that gives up sets bit 1 of the handle's
// status word and lets the CTA run to its end, where the tensor memory is released.
#include <cuda.h>   // CUtensorMap and its enums; the encode function itself is looked up at run time

#include "kvr_internal.h"

namespace {

constexpr int TC_THREADS = 320;
constexpr int TC_NT = 128;                      // keys per tile
constexpr int TC_STAGES = 2;
constexpr int TC_HALF_BYTES = 128 * 128;        // one swizzle atom column: 128 rows x 128 bytes
constexpr int TC_TILE_BYTES = 2 * TC_HALF_BYTES;
constexpr int TC_TMEM_COLS = 256;
constexpr int TC_DYN_SMEM = (1 + TC_STAGES) * TC_TILE_BYTES + 1024;   // Q + ring + alignment slack
constexpr unsigned FULL = 0xFFFFFFFFu;

// barrier indices
constexpr int B_Q = 0, B_FULL = 1, B_EMPTY = B_FULL + TC_STAGES, B_TFULL = B_EMPTY + TC_STAGES, B_TEMPTY = B_TFULL + 2,
              B_EPI = B_TEMPTY + 2, B_COUNT = B_EPI + 1;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n"
        " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        " selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t0));
    while (!mbar_try_wait(bar, parity)) {
        asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
        if (t - t0 > limit_ns) return false;
    }
    return true;
}
// One box of 64 elements x 128 rows (16 KB) -> shared memory; x is 0 or 64 (a multiple of 16 bytes).
__device__ __forceinline__ void tma_load_2d(uint32_t sdst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n"
                 ::"r"(sdst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}
// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024
// bytes apart (stride byte offset), descriptor version 1, leading byte offset unused (1).
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
        " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];\n"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
// the values of earlier tmem_ld32 calls may be used after this
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory"); }
__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// v[c] of lane r = element (row r, column c) of a 32 x 32 block; afterwards v[0] of lane c is the
// sum of column c over the 32 rows (fixed order of additions).
template <int OFF>
__device__ __forceinline__ void col_sum_step(float (&v)[32], int lane) {
    const bool hi = (lane & OFF) != 0;
#pragma unroll
    for (int i = 0; i < OFF; ++i) {
        const float keep = hi ? v[i + OFF] : v[i];
        const float send = hi ? v[i] : v[i + OFF];
        v[i] = keep + __shfl_xor_sync(FULL, send, OFF);
    }
}

template <typename T> struct UmmaFmt;
template <> struct UmmaFmt<__half> { static constexpr uint32_t v = 0; };
template <> struct UmmaFmt<__nv_bfloat16> { static constexpr uint32_t v = 1; };

template <typename T, int PASS>
__global__ void __launch_bounds__(TC_THREADS, 2)
score_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, int N, int M,
                int W, int causal, int chunk, int n_chunks, float scale_log2e,
                float2* partial /*[u][2 n_chunks][Mpad]: written by pass 1, read by pass 2*/,
                float* __restrict__ scores_all, int max_ctx, int inst0, int* __restrict__ status,
                unsigned long long wait_ns /*limit of every mbarrier wait*/,
                uint32_t tx_extra /*0; a test announces bytes that never arrive, so that the waits run out*/) {
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[B_COUNT];
    __shared__ uint32_t s_tmem;
    __shared__ float s_col[2][4][TC_NT];
    __shared__ float2 s_stat[2][128];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int u = blockIdx.y, ck = blockIdx.x;
    kvr_pdl_trigger();         // the next kernel of the compress may take over SMs as they become free
    const int m_tiles = (M + 127) / 128, Mpad = m_tiles * 128;
    const int n_begin = ck * chunk, n_end = min(n_begin + chunk, N);
    const int n_tiles = (n_end - n_begin + TC_NT - 1) / TC_NT;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;     // the swizzle pattern repeats every 1024 bytes
    const uint32_t sQ = base, sK = base + TC_TILE_BYTES;
    const uint32_t bar0 = smem_u32(s_bar);
    auto bar = [&](int i) { return bar0 + 8u * (uint32_t)i; };

    if (tid == 0) {
        mbar_init(bar(B_Q), 1);
        for (int s = 0; s < TC_STAGES; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(bar(B_TFULL + i), 1); mbar_init(bar(B_TEMPTY + i), 8); }
        mbar_init(bar(B_EPI), 8);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n" ::"r"(smem_u32(&s_tmem)), "r"(TC_TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *reinterpret_cast<volatile uint32_t*>(&s_tmem);

    // instruction descriptor: fp32 accumulator, A and B of type T, both K-major, N = 128, M = 128
    constexpr uint32_t idesc = (1u << 4) | (UmmaFmt<T>::v << 7) | (UmmaFmt<T>::v << 10) | ((uint32_t)(TC_NT >> 3) << 17) | ((128u >> 4) << 24);
    float* sc = scores_all + (size_t)(inst0 + u) * max_ctx;
    bool gave_up = false;
    uint32_t epi_round = 0;

    for (int mt = 0; mt < m_tiles; ++mt) {
        const uint32_t it0 = (uint32_t)mt * (uint32_t)n_tiles;           // tiles consumed before this m-tile
        if (warp == 0) {
            if (lane == 0 && !gave_up) {
                mbar_expect_tx(bar(B_Q), TC_TILE_BYTES + tx_extra);
                tma_load_2d(sQ, &tmQ, 0, u * M + mt * 128, bar(B_Q));
                tma_load_2d(sQ + TC_HALF_BYTES, &tmQ, 64, u * M + mt * 128, bar(B_Q));
                for (int i = 0; i < n_tiles; ++i) {
                    const uint32_t it = it0 + i, s = it % TC_STAGES, ph = (it / TC_STAGES) & 1u;
                    if (!mbar_wait(bar(B_EMPTY + s), ph ^ 1u, wait_ns)) { gave_up = true; break; }
                    mbar_expect_tx(bar(B_FULL + s), TC_TILE_BYTES);
                    const int row = u * N + n_begin + i * TC_NT;
                    tma_load_2d(sK + s * TC_TILE_BYTES, &tmK, 0, row, bar(B_FULL + s));
                    tma_load_2d(sK + s * TC_TILE_BYTES + TC_HALF_BYTES, &tmK, 64, row, bar(B_FULL + s));
                }
            }
        } else if (warp == 1) {
            if (lane == 0 && !gave_up) {
                if (!mbar_wait(bar(B_Q), (uint32_t)mt & 1u, wait_ns)) gave_up = true;
                for (int i = 0; i < n_tiles && !gave_up; ++i) {
                    const uint32_t it = it0 + i, s = it % TC_STAGES, ph = (it / TC_STAGES) & 1u;
                    const uint32_t buf = it & 1u, bph = (it >> 1) & 1u;
                    if (!mbar_wait(bar(B_TEMPTY + buf), bph ^ 1u, wait_ns) || !mbar_wait(bar(B_FULL + s), ph, wait_ns)) { gave_up = true; break; }
                    tc_fence_after();
#pragma unroll
                    for (int k = 0; k < 8; ++k) {                       // 8 x 16 channels = the head dimension
                        const uint32_t off = (uint32_t)(k >> 2) * TC_HALF_BYTES + (uint32_t)(k & 3) * 32u;
                        umma_f16(tmem + buf * TC_NT, umma_desc(sQ + off), umma_desc(sK + s * TC_TILE_BYTES + off), idesc, k > 0);
                    }
                    umma_commit(bar(B_EMPTY + s));        // the key tile may be overwritten once these MMAs have read it
                    umma_commit(bar(B_TFULL + buf));      // the accumulator is complete
                }
            }
        } else {
            const int q = warp & 3, half = (warp - 2) >> 2;
            const int row = mt * 128 + q * 32 + lane;
            const bool row_ok = row < M;
            const bool rows_inside = mt * 128 + 128 <= M;                // (uniform) no row of the tile is padding
            // keys this row may see: all N, or (observation window inside the context) up to its own position
            const int n_vis = causal ? N - W + 1 + (row % W) : N;
            const int n_free = causal ? N - W + 1 : N;                   // keys below this index are visible to every row
            float m_run = -INFINITY, l_run = 0.f;
            if (PASS == 2) {
                // Final maximum and reciprocal sum of this row from the (max, sum) pairs pass 1 left per
                // chunk half.  The two threads that share a row (one per column half) fold every other
                // pair each, 16 loads in flight, then exchange through shared memory; both add the two
                // halves in the same order, so they hold identical statistics.  (Every CTA of the
                // head-instance repeats this while its first key tiles are on their way.)
                // (pass 2 is launched as a programmatic dependent of pass 1: its loads and its first tiles
                // run beside pass 1's last CTAs; what pass 1 wrote is needed from here on)
                kvr_pdl_wait();
                const float2* pp = partial + (size_t)u * 2 * n_chunks * Mpad + row;
                const int n_parts = 2 * n_chunks;
                float mx = -INFINITY, l = 0.f;
                for (int c0 = half; c0 < n_parts; c0 += 32) {
                    float2 x[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j)
                        x[j] = (c0 + 2 * j < n_parts) ? __ldcg(pp + (size_t)(c0 + 2 * j) * Mpad) : make_float2(-INFINITY, 0.f);
                    float mn = mx;
#pragma unroll
                    for (int j = 0; j < 16; ++j) mn = fmaxf(mn, x[j].x);
                    if (mn > -INFINITY) {
                        l *= ex2f(mx - mn);
#pragma unroll
                        for (int j = 0; j < 16; ++j) l += (x[j].y > 0.f) ? x[j].y * ex2f(x[j].x - mn) : 0.f;
                        mx = mn;
                    }
                }
                s_stat[half][q * 32 + lane] = make_float2(mx, l);
                __threadfence_block();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_EPI));
                if (!__all_sync(FULL, mbar_wait(bar(B_EPI), epi_round & 1u, wait_ns))) gave_up = true;
                ++epi_round;
                const float2 a0 = s_stat[0][q * 32 + lane], a1 = s_stat[1][q * 32 + lane];
                const float mrow = fmaxf(a0.x, a1.x);                    // finite: every row has seen column 0
                const float lrow = a0.y * ex2f(a0.x - mrow) + a1.y * ex2f(a1.x - mrow);
                float lg;
                asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(lg) : "f"(lrow));
                m_run = mrow + lg;                                       // exp2(s - m_run) = exp2(s - max) / sum
            }
            for (int i = 0; i < n_tiles && !gave_up; ++i) {
                const uint32_t it = it0 + i, buf = it & 1u, bph = (it >> 1) & 1u;
                if (!__all_sync(FULL, mbar_wait(bar(B_TFULL + buf), bph, wait_ns))) { gave_up = true; break; }
                tc_fence_after();
                const int n0 = n_begin + i * TC_NT;
                float vv[2][32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + buf * TC_NT + (uint32_t)(half * 64), vv[0]);
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + buf * TC_NT + (uint32_t)(half * 64 + 32), vv[1]);
                tmem_ld_wait();
                tc_fence_before();                                       // this warp has read its part of the buffer
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_TEMPTY + buf));
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {
                    const int col0 = n0 + half * 64 + blk * 32;
                    float (&v)[32] = vv[blk];
                    if (col0 >= N) continue;                             // (uniform) nothing valid in this block
                    const bool inside = col0 + 32 <= n_free;             // (uniform) no column of the block is masked
                    if (PASS == 1) {
                        // maximum of the raw dot products first (the scale is positive), then one
                        // multiply-add and one exponential per element
                        if (!inside) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) v[c] = (col0 + c < n_vis) ? v[c] : -INFINITY;
                        }
                        float tm = v[0];
#pragma unroll
                        for (int c = 1; c < 32; ++c) tm = fmaxf(tm, v[c]);
                        if (tm == -INFINITY) continue;                    // this row sees no key of the block
                        const float mn = fmaxf(m_run, tm * scale_log2e);
                        float add = 0.f;
#pragma unroll
                        for (int c = 0; c < 32; ++c) add += ex2f(fmaf(v[c], scale_log2e, -mn));
                        l_run = l_run * ex2f(m_run - mn) + add;
                        m_run = mn;
                    } else {
                        // m_run = row maximum + log2(row sum): the exponential is the normalised probability
#pragma unroll
                        for (int c = 0; c < 32; ++c) v[c] = ex2f(fmaf(v[c], scale_log2e, -m_run));
                        if (!inside || !rows_inside) {
#pragma unroll
                            for (int c = 0; c < 32; ++c) v[c] = (row_ok && col0 + c < n_vis) ? v[c] : 0.f;
                        }
                        col_sum_step<16>(v, lane);
                        col_sum_step<8>(v, lane);
                        col_sum_step<4>(v, lane);
                        col_sum_step<2>(v, lane);
                        col_sum_step<1>(v, lane);
                        s_col[it & 1u][q][half * 64 + blk * 32 + lane] = v[0];
                    }
                }
                if (PASS == 2) {
                    // the four row quarters of a column are added by one thread, in a fixed order
                    __threadfence_block();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_EPI));
                    if (!__all_sync(FULL, mbar_wait(bar(B_EPI), epi_round & 1u, wait_ns))) { gave_up = true; break; }
                    ++epi_round;
                    const int et = tid - 64;
                    if (et < TC_NT) {
                        const int col = n0 + et;
                        if (col < N) {
                            const float tot = ((s_col[it & 1u][0][et] + s_col[it & 1u][1][et]) + s_col[it & 1u][2][et]) + s_col[it & 1u][3][et];
                            sc[col] = (mt == 0) ? tot : sc[col] + tot;
                        }
                    }
                }
            }
            if (PASS == 1 && !gave_up)
                partial[((size_t)u * 2 * n_chunks + 2 * ck + half) * Mpad + row] = make_float2(m_run, l_run);
        }
        if (gave_up) atomicOr(status, 2);
        tc_fence_before();
        __syncthreads();          // every tile of this m-tile is consumed: Q and the ring are idle
        tc_fence_after();
    }
    if (warp == 1)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" ::"r"(tmem), "r"(TC_TMEM_COLS) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            p = nullptr;
        return (EncodeTiledFn)p;
    }();
    return fn;
}

// rows x 128 elements of 2 bytes, boxes of 64 elements x 128 rows, 128-byte swizzle, zeros out of range
bool make_map(CUtensorMap* tm, const void* ptr, uint64_t rows, bool bf16) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)KVR_D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)KVR_D * 2};
    const cuuint32_t box[2] = {64, 128};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr),
              dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T>
cudaError_t launch_typed(kvr_sketch* sk, const ScoreShape& s, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                         cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(score_tc_kernel<T, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_DYN_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(score_tc_kernel<T, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_DYN_SMEM);
    if (e != cudaSuccess) return e;
    float2* partial = (float2*)sk->ws_score;
    dim3 grid(s.n_chunks, s.n_inst);
    score_tc_kernel<T, 1><<<grid, TC_THREADS, TC_DYN_SMEM, st>>>(tmQ, tmK, s.N, s.M, s.W, s.causal, s.chunk, s.n_chunks, s.scale_log2e,
                                                                 partial, sk->scores, sk->d.max_context,
                                                                 s.inst0, sk->dev_status, sk->wait_ns, sk->tx_extra);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    e = kvr_launch_after(score_tc_kernel<T, 2>, grid, dim3(TC_THREADS), TC_DYN_SMEM, st, true, tmQ, tmK, s.N, s.M, s.W, s.causal,
                         s.chunk, s.n_chunks, s.scale_log2e, partial, sk->scores, sk->d.max_context, s.inst0, sk->dev_status,
                         sk->wait_ns, sk->tx_extra);
    sk->launches += 2;
    return e;
}

}  // namespace

// The tensor-memory path takes every shape whose two operands are at least one box high (128 rows
// in total) and 16-byte aligned; smaller problems stay on the mma.sync kernels.
bool kvr_scores_tc_supported(const ScoreShape& s, const void* K, const void* Q) {
    if ((long long)s.n_inst * s.N < 128 || (long long)s.n_inst * s.M < 128) return false;
    if (((uintptr_t)K | (uintptr_t)Q) & 15u) return false;
    return encode_fn() != nullptr;
}

// Keys per CTA (a multiple of the 128-key tile) so that about two CTAs per SM are launched.
void kvr_scores_tc_plan(const kvr_sketch* sk, ScoreShape* s) {
    int want = (2 * sk->n_sm) / s->n_inst;
    if (want < 1) want = 1;
    int chunk = (s->N + want - 1) / want;
    chunk = ((chunk + TC_NT - 1) / TC_NT) * TC_NT;
    s->chunk = chunk;
    s->n_chunks = (s->N + chunk - 1) / chunk;
}

size_t kvr_scores_tc_ws_bytes(const ScoreShape& s) {
    const int Mpad = ((s.M + 127) / 128) * 128;
    return sizeof(float2) * ((size_t)s.n_inst * 2 * s.n_chunks * Mpad);
}

// Workspace: partial [n_inst][2 n_chunks][Mpad] float2.
cudaError_t kvr_launch_scores_tc(kvr_sketch* sk, const ScoreShape& s, const void* K, const void* Q, cudaStream_t st) {
    CUtensorMap tmQ, tmK;
    const bool bf16 = sk->d.kv_dtype == KVR_BF16;
    if (!make_map(&tmQ, Q, (uint64_t)s.n_inst * s.M, bf16) || !make_map(&tmK, K, (uint64_t)s.n_inst * s.N, bf16))
        return cudaErrorInvalidValue;
    if (bf16) return launch_typed<__nv_bfloat16>(sk, s, tmQ, tmK, st);
    return launch_typed<__half>(sk, s, tmQ, tmK, st);
}
