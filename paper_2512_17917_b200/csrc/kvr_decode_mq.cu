// Decode attention for several queries per head over the mixed cache (speculative / chunked decoding):
// Algorithm 4 (Revive) fused with p = Softmax(q K^T / sqrt(d_k)), out = p V of the Calculation Phase,
// where the cost of Algorithm 2's reconstruction is shared by all queries.
//
// Up to 64 query rows (query heads of one kv head x queries) are served per launch, 16 per warp: the
// warps of a CTA form teams of MT = 1, 2 or 4 that share one tile of reconstructed tokens (each
// warp reconstructs its part of the tile, then runs the contractions for its own 16 rows), so a
// token is reconstructed once for all rows of the launch.  As in the staged
// single-query kernel, a CTA serves (a slice of) one class of compressed tokens with the class's
// row-1 and row-2 cells staged in shared memory, and a group of 16 lanes reconstructs one token at a
// time (8 channels per lane, the row-0 cell of the current run in registers).  What differs is what
// happens to a reconstructed vector: instead of feeding dot products of one query group, it is split
// into two 16-bit floats (hi + lo, 22 significant bits) and written to a small per-warp tile, and the
// two contractions run on the tensor cores with fp32 accumulation:
//     S[16 x 8]   = Q[16 x 128] . (K~hi + K~lo)^T          (mma m16n8k16, 2 x 8 per tile)
//     O[16 x 128] += (Phi + Plo)[16 x 8] . (V~hi + V~lo)    (mma m16n8k8, hi.hi + hi.lo + lo.hi)
// with an online softmax per warp in between (running maximum raised only when exceeded by 2^8, so
// that the weights stay inside the 16-bit range).  Retained rows (exact 16-bit keys and values) go
// through the same tiles without a lo part.  Every warp walks its own tokens; warps meet only for the
// CTA's record, and the last CTA of a head-instance to arrive merges the records (nobody waits).
#include <cuda_fp16.h>

#include "kvr_decode_common.cuh"

namespace {
using namespace kvr_dec;

constexpr int MQ_THREADS = 256, MQ_WARPS = MQ_THREADS / 32, MQ_GROUPS = 2 * MQ_WARPS;
constexpr int MQ_ROWS = 16;                    // query rows per launch
constexpr int MQ_TILE = 8;                     // tokens per tile
constexpr int MQ_PITCH = 272;                  // bytes of a tile row: 128 x 16 bit + 16 (conflict-free 8 x 8 matrix loads)
constexpr int MQ_TILE_BYTES = MQ_TILE * MQ_PITCH;
constexpr int MQ_CELLB = 2 * KVR_D * 4, MQ_HALFB = KVR_D * 4;
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr float MQ_GAP = 8.f;
constexpr size_t MQ_SMEM_LIMIT = 227 * 1024 - 1024;

struct MqParams {
    const void* q;          // [n_inst][M][128] 16-bit, M = query rows per head-instance
    const uint2* Kr;        // [n_inst][R][32]
    const uint2* Vr;
    const float* cells;     // handle base: [inst][2][r][b][128]
    const uint2* clist;     // handle base: [inst][max_ctx]
    const int32_t* coff;    // handle base: [inst][C*C+1]
    float* part;            // [n_inst][records][16][PART]
    uint32_t* tickets;      // handle base: [inst]
    float* out;             // [n_inst][M][128]
    int* status;
    int inst0, R, b, C, logC, n1, max_ctx, S, lcap;
    int M, row0, Qn, causal;    // rows per head-instance, first row of this launch, queries per head, mask
    uint32_t zero;
    float scale_log2e;
};

struct MqLayout {
    int ctrl, ring, tiles, list, cells, total;
};
__host__ __device__ inline MqLayout mq_layout(int n1, int lcap) {
    MqLayout L;
    int o = 0;
    L.ctrl = o;  o += 32;                                  // last-arriver flag; staging mbarriers at +16, +24
    L.ring = o;  o += MQ_GROUPS * 2 * MQ_HALFB;            // per group: key half and value half of a row-0 cell in flight
    L.tiles = o; o += MQ_WARPS * 2 * MQ_TILE_BYTES;        // per team of MT warps: hi tile, lo tile of 8 MT tokens
    L.list = o;  o += ((lcap + 2) * 8 + 15) & ~15;
    L.cells = o; o += 2 * n1 * MQ_CELLB;                   // row-1 slice, row-2 slice (later: the warps' records)
    L.total = o;
    if (L.total - L.cells < MQ_WARPS * MQ_ROWS * PART * 4) L.total = L.cells + MQ_WARPS * MQ_ROWS * PART * 4;
    return L;
}

__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(gsrc));
}
__device__ __forceinline__ float4 lds128(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 e;
    asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];\n" : "=r"(e.x), "=r"(e.y) : "r"(addr) : "memory");
    return e;
}
__device__ __forceinline__ void sts64(uint32_t addr, uint32_t a, uint32_t b) {
    asm volatile("st.shared.v2.u32 [%0], {%1,%2};\n" ::"r"(addr), "r"(a), "r"(b) : "memory");
}
__device__ __forceinline__ void mq_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
__device__ __forceinline__ void mq_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mq_bulk_g2s(uint32_t sdst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(sdst), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ bool mq_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n"
        " mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        " selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait (0.2 s), as in the staged kernel: gives up instead of hanging
__device__ __forceinline__ bool mq_wait(uint32_t bar, uint32_t parity) {
    if (mq_try_wait(bar, parity)) return true;
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t0));
    while (!mq_try_wait(bar, parity)) {
        asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
        if (t - t0 > 200ull * 1000 * 1000) return false;
    }
    return true;
}
// four 8 x 8 matrices of 16-bit elements; lane l supplies the address of row l % 8 of matrix l / 8
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm4_t(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma_k16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ uint32_t pack_h2(float lo, float hi) {
    const __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
// x = hi + lo with hi, lo 16-bit floats (hi = x rounded, lo = the rest rounded): 22 significant bits
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
    const __half2 h = __floats2half2_rn(x0, x1);
    const float2 hf = __half22float2(h);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = pack_h2(x0 - hf.x, x1 - hf.y);
}
// 16-bit pair of the cache type -> 16-bit float pair (bf16 values fit: 8 significant bits)
template <typename T>
__device__ __forceinline__ uint32_t to_h2(uint32_t u) {
    if constexpr (std::is_same<T, __half>::value) return u;
    else {
        const float2 f = KvrType<T>::to_f2(u);
        return pack_h2(f.x, f.y);
    }
}

template <typename T, int MT>
__global__ void __launch_bounds__(MQ_THREADS, 1)
decode_mq_kernel(const MqParams p) {
    constexpr int TPH = 4;                              // tokens a group of 16 lanes reconstructs per tile
    constexpr int TT = MQ_TILE * MT;                    // tokens of a team's tile: every warp fills 8 slots of it
    constexpr uint32_t TEAM_TILE_BYTES = (uint32_t)MT * MQ_TILE_BYTES;
    constexpr int NTEAMS = MQ_WARPS / MT, ROWS_L = MQ_ROWS * MT;
    extern __shared__ __align__(16) unsigned char smem[];
    const MqLayout L = mq_layout(p.n1, p.lcap);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, gw = lane >> 4, lg = lane & 15;
    const int grp = warp * 2 + gw;
    const int team = warp / MT, wt = warp % MT, hw = wt * 2 + gw;      // team, warp in team (= its 16 rows), group in team
    const int rowbase = p.row0 + wt * MQ_ROWS;
    auto team_sync = [&]() {
        if constexpr (MT == 1) __syncwarp();
        else asm volatile("bar.sync %0, %1;\n" ::"r"(1 + team), "r"(32 * MT) : "memory");
    };
    const int fg = lane >> 2, ft = lane & 3;             // fragment coordinates: row group, column pair
    const int u = blockIdx.y, inst = p.inst0 + u, b = p.b, C = p.C, n1 = p.n1;
    const int rec = blockIdx.x, n_rec = gridDim.x;
    const int cls = rec / p.S, sp = rec - cls * p.S;
    const int ci = cls >> p.logC, cj = cls & (C - 1);
    int k_lo, k_hi;
    {
        const int32_t* coff = p.coff + (size_t)inst * (C * C + 1);
        k_lo = __ldg(coff + cls);
        k_hi = __ldg(coff + cls + 1);
    }
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t cells_s = smem_s + L.cells, list_base = smem_s + L.list;
    const uint32_t bar_cells = smem_s + L.ctrl + 16u, bar_list = smem_s + L.ctrl + 24u;
    const float* cellsK = p.cells + (size_t)inst * 2 * KVR_R * b * KVR_D;
    const float* cellsV = cellsK + (size_t)KVR_R * b * KVR_D;
    // ---------------------------------------------------------------- staging (as in the staged kernel)
    if (tid == 0) {
        mq_mbar_init(bar_cells, 1);
        mq_mbar_init(bar_list, 1);
        const int cnt1 = (b - ci + C - 1) >> p.logC, cnt2 = (b - cj + C - 1) >> p.logC;
        mq_expect_tx(bar_cells, (uint32_t)((cnt1 + cnt2) * MQ_CELLB));
    }
    __syncthreads();
    for (int i = warp + lane * MQ_WARPS; i < 4 * n1; i += MQ_THREADS) {
        const int idx = i >> 1, kv = i & 1;
        const int h = (idx < n1) ? idx * C + ci : (idx - n1) * C + cj;
        const int row = (idx < n1) ? 1 : 2;
        if (h < b)
            mq_bulk_g2s(cells_s + (uint32_t)(idx * MQ_CELLB + kv * MQ_HALFB),
                        (kv ? cellsV : cellsK) + ((size_t)row * b + h) * KVR_D, MQ_HALFB, bar_cells);
    }
    const int k_len = k_hi - k_lo;
    const int s_begin = k_lo + (int)((long long)k_len * sp / p.S), s_end = k_lo + (int)((long long)k_len * (sp + 1) / p.S);
    const int r_begin = (int)((long long)p.R * rec / n_rec), r_end = (int)((long long)p.R * (rec + 1) / n_rec);
    const uint2* clist = p.clist + (size_t)inst * p.max_ctx;
    const int lcap = p.lcap, len0 = min(lcap, s_end - s_begin);
    const int lshift = (int)(((size_t)inst * p.max_ctx + s_begin) & 1);
    if (len0 > 0 && tid == 0) {
        const uint32_t bytes = (uint32_t)(((len0 + lshift + 1) & ~1) * 8);
        mq_expect_tx(bar_list, bytes);
        mq_bulk_g2s(list_base, clist + (s_begin - lshift), bytes, bar_list);
    }

    // ---------------------------------------------------------------- the queries: A fragments of the 16
    // rows of this launch (rows beyond the head-instance's M are zero), natural channel order
    uint32_t qa[8][4];
    {
        const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q) + ((size_t)u * p.M + rowbase) * (KVR_D / 2);
        const bool v0 = rowbase + fg < p.M, v1 = rowbase + fg + 8 < p.M;
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            qa[s][0] = v0 ? to_h2<T>(__ldg(q32 + (size_t)fg * 64 + 8 * s + ft)) : 0u;
            qa[s][1] = v1 ? to_h2<T>(__ldg(q32 + (size_t)(fg + 8) * 64 + 8 * s + ft)) : 0u;
            qa[s][2] = v0 ? to_h2<T>(__ldg(q32 + (size_t)fg * 64 + 8 * s + 4 + ft)) : 0u;
            qa[s][3] = v1 ? to_h2<T>(__ldg(q32 + (size_t)(fg + 8) * 64 + 8 * s + 4 + ft)) : 0u;
        }
    }
    // rows of the storage a query row may see (the mask among the queries' own tokens)
    int vis[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int r = rowbase + fg + 8 * h;
        const int t = r % p.Qn;
        vis[h] = p.causal ? p.R - p.Qn + t + 1 : p.R;
    }
    float m_run[2] = {M_EMPTY, M_EMPTY}, l_run[2] = {0.f, 0.f};
    float O[16][4];
#pragma unroll
    for (int nt = 0; nt < 16; ++nt)
#pragma unroll
        for (int k = 0; k < 4; ++k) O[nt][k] = 0.f;

    const uint32_t tile_hi = smem_s + L.tiles + (uint32_t)team * 2u * TEAM_TILE_BYTES, tile_lo = tile_hi + TEAM_TILE_BYTES;
    // this lane's row address for the 8 x 8 matrix loads (matrix lane / 8, row lane % 8)
    const uint32_t ldsm_off = (uint32_t)((lane & 7) * MQ_PITCH + (lane >> 3) * 16);

    // S = Q K^T over the tile (hi, and lo when the tile has one), softmax step, weights as A fragments.
    // live: bit s set = tile slot s holds a token; row_base >= 0: slot s is row row_base + s of the
    // storage (a retained row: the mask among the queries' own tokens applies), else a compressed token.
    uint32_t pa_hi[MT][2], pa_lo[MT][2];                  // per 8 tokens: rows fg | fg + 8, columns 2 ft, 2 ft + 1
    auto qk_softmax = [&](bool with_lo, unsigned live, int row_base) {
        float c[MT][4];
#pragma unroll
        for (int nt = 0; nt < MT; ++nt) {
            c[nt][0] = c[nt][1] = c[nt][2] = c[nt][3] = 0.f;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t r[4];
                ldsm4(tile_hi + (uint32_t)(nt * MQ_TILE_BYTES) + ldsm_off + j * 64, r);
                mma_k16(c[nt], qa[2 * j], r[0], r[1]);
                mma_k16(c[nt], qa[2 * j + 1], r[2], r[3]);
            }
            if (with_lo) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t r[4];
                    ldsm4(tile_lo + (uint32_t)(nt * MQ_TILE_BYTES) + ldsm_off + j * 64, r);
                    mma_k16(c[nt], qa[2 * j], r[0], r[1]);
                    mma_k16(c[nt], qa[2 * j + 1], r[2], r[3]);
                }
            }
        }
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nt = 0; nt < MT; ++nt)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int col = 8 * nt + 2 * ft + (k & 1), h = k >> 1;
                const bool ok = ((live >> col) & 1u) && (row_base < 0 || row_base + col < vis[h]);
                c[nt][k] = ok ? c[nt][k] * p.scale_log2e : -INFINITY;
                mx[h] = fmaxf(mx[h], c[nt][k]);
            }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(FULL, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(FULL, mx[h], 2));
        }
        const bool g0 = mx[0] > m_run[0] + MQ_GAP, g1 = mx[1] > m_run[1] + MQ_GAP;
        if (__any_sync(FULL, g0 || g1)) {
            const float n0 = g0 ? mx[0] : m_run[0], n1_ = g1 ? mx[1] : m_run[1];
            const float c0 = ex2(m_run[0] - n0), c1 = ex2(m_run[1] - n1_);
            l_run[0] *= c0;
            l_run[1] *= c1;
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) { O[nt][0] *= c0; O[nt][1] *= c0; O[nt][2] *= c1; O[nt][3] *= c1; }
            m_run[0] = n0;
            m_run[1] = n1_;
        }
#pragma unroll
        for (int nt = 0; nt < MT; ++nt) {
            float pr[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) pr[k] = ex2(c[nt][k] - m_run[k >> 1]);
            l_run[0] += pr[0] + pr[1];
            l_run[1] += pr[2] + pr[3];
            split2(pr[0], pr[1], pa_hi[nt][0], pa_lo[nt][0]);
            split2(pr[2], pr[3], pa_hi[nt][1], pa_lo[nt][1]);
        }
    };
    // O += P V over the tile: 8 tokens per multiply (MT = 1) or 16 (two adjacent groups of 8 form the
    // k dimension: their weight fragments are the four A registers as they stand)
    auto pv = [&](bool with_lo) {
        if constexpr (MT == 1) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                uint32_t r[4];
                ldsm4_t(tile_hi + ldsm_off + j * 64, r);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    mma_k8(O[4 * j + i], pa_hi[0][0], pa_hi[0][1], r[i]);
                    mma_k8(O[4 * j + i], pa_lo[0][0], pa_lo[0][1], r[i]);
                }
            }
            if (with_lo) {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t r[4];
                    ldsm4_t(tile_lo + ldsm_off + j * 64, r);
#pragma unroll
                    for (int i = 0; i < 4; ++i) mma_k8(O[4 * j + i], pa_hi[0][0], pa_hi[0][1], r[i]);
                }
            }
        } else {
#pragma unroll
            for (int ks = 0; ks < MT / 2; ++ks) {
                const uint32_t ah[4] = {pa_hi[2 * ks][0], pa_hi[2 * ks][1], pa_hi[2 * ks + 1][0], pa_hi[2 * ks + 1][1]};
                const uint32_t al[4] = {pa_lo[2 * ks][0], pa_lo[2 * ks][1], pa_lo[2 * ks + 1][0], pa_lo[2 * ks + 1][1]};
                const uint32_t t0 = (uint32_t)(2 * ks * MQ_TILE_BYTES) + ldsm_off, t1 = t0 + MQ_TILE_BYTES;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t r0[4], r1[4];
                    ldsm4_t(tile_hi + t0 + j * 64, r0);
                    ldsm4_t(tile_hi + t1 + j * 64, r1);
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        mma_k16(O[4 * j + i], ah, r0[i], r1[i]);
                        mma_k16(O[4 * j + i], al, r0[i], r1[i]);
                    }
                }
                if (with_lo) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        uint32_t r0[4], r1[4];
                        ldsm4_t(tile_lo + t0 + j * 64, r0);
                        ldsm4_t(tile_lo + t1 + j * 64, r1);
#pragma unroll
                        for (int i = 0; i < 4; ++i) mma_k16(O[4 * j + i], ah, r0[i], r1[i]);
                    }
                }
            }
        }
    };

    // ---------------------------------------------------------------- retained rows (exact keys, values)
    {
        const int n = r_end - r_begin, per = (n + NTEAMS - 1) / NTEAMS;
        const int w0 = r_begin + min(team * per, n), w1 = r_begin + min((team + 1) * per, n);
        const uint2* Kr = p.Kr + (size_t)u * p.R * 32 + lg;
        const uint2* Vr = p.Vr + (size_t)u * p.R * 32 + lg;
        for (int base = w0; base < w1; base += TT) {
            const int nl = min(TT, w1 - base);
            const unsigned live = nl >= 32 ? 0xFFFFFFFFu : (1u << nl) - 1u;
            uint2 x[TPH][2];
#pragma unroll
            for (int it = 0; it < TPH; ++it) {
                const int slot = 8 * wt + 2 * it + gw, row = base + (slot < nl ? slot : 0);
                x[it][0] = Kr[(size_t)row * 32];
                x[it][1] = Kr[(size_t)row * 32 + 16];
            }
#pragma unroll
            for (int it = 0; it < TPH; ++it) {
                const uint32_t dst = tile_hi + (uint32_t)((8 * wt + 2 * it + gw) * MQ_PITCH + lg * 8);
                sts64(dst, to_h2<T>(x[it][0].x), to_h2<T>(x[it][0].y));
                sts64(dst + 128, to_h2<T>(x[it][1].x), to_h2<T>(x[it][1].y));
            }
#pragma unroll
            for (int it = 0; it < TPH; ++it) {                   // the values are on their way while the keys are used
                const int slot = 8 * wt + 2 * it + gw, row = base + (slot < nl ? slot : 0);
                x[it][0] = Vr[(size_t)row * 32];
                x[it][1] = Vr[(size_t)row * 32 + 16];
            }
            team_sync();
            qk_softmax(false, live, base);
            team_sync();
#pragma unroll
            for (int it = 0; it < TPH; ++it) {
                const uint32_t dst = tile_hi + (uint32_t)((8 * wt + 2 * it + gw) * MQ_PITCH + lg * 8);
                sts64(dst, to_h2<T>(x[it][0].x), to_h2<T>(x[it][0].y));
                sts64(dst + 128, to_h2<T>(x[it][1].x), to_h2<T>(x[it][1].y));
            }
            team_sync();
            pv(false);
            team_sync();
        }
    }

    // ---------------------------------------------------------------- compressed tokens
    const uint32_t ringK = smem_s + L.ring + (uint32_t)(grp * 2 * MQ_HALFB + lg * 16), ringV = ringK + MQ_HALFB;
    const float* g0K = cellsK + 4 * lg;
    const float* g0V = cellsV + 4 * lg;
    auto fetch_half = [&](uint32_t dst, const float* g0, uint32_t c0, uint32_t z) {
        const float* g = g0 + (size_t)c0 * KVR_D;
        cp_async16(dst + z, g);
        cp_async16(dst + z + 256, g + 64);
        asm volatile("cp.async.commit_group;\n" ::);
    };
    // take the fetched half cell into registers, ask for the next run's (the copy's address depends
    // on the loaded values, so that it cannot start before they are read; z is always 0)
    auto switch_run = [&](float (&r0v)[8], uint32_t ring, const float* g0, uint32_t c0_next) {
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        const float4 a = lds128(ring), c = lds128(ring + 256);
        r0v[0] = a.x; r0v[1] = a.y; r0v[2] = a.z; r0v[3] = a.w;
        r0v[4] = c.x; r0v[5] = c.y; r0v[6] = c.z; r0v[7] = c.w;
        fetch_half(ring, g0, c0_next, (__float_as_uint(a.w) | __float_as_uint(c.w)) & p.zero);
    };
    const uint32_t lane_cells = cells_s + (uint32_t)(lg * 16);
    if (!mq_wait(bar_cells, 0)) atomicOr(p.status, 1);
    for (int cb = s_begin, st = 0; cb < s_end; cb += lcap, ++st) {
        const int len = min(lcap, s_end - cb);
        const uint32_t list_s = list_base + (uint32_t)(st == 0 ? lshift : 0) * 8u;
        if (st == 0) {
            if (!mq_wait(bar_list, 0)) atomicOr(p.status, 1);
        } else {
            __syncthreads();
            uint2* s_list = reinterpret_cast<uint2*>(smem + L.list);
            for (int i = tid; i < len; i += MQ_THREADS) s_list[i] = clist[cb + i];
            __syncthreads();
        }
        // the team's tokens, one contiguous part per group of 16 lanes (2 MT groups)
        const int per = (len + NTEAMS - 1) / NTEAMS;
        const int w0 = min(team * per, len), w1 = min((team + 1) * per, len);
        const int half = (w1 - w0 + 2 * MT - 1) / (2 * MT);                  // tokens per group (the last groups may have fewer)
        const int g_begin = w0 + min(hw * half, w1 - w0), g_cnt = min(half, w1 - w0 - min(hw * half, w1 - w0));
        float k0[8], v0[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) { k0[x] = 0.f; v0[x] = 0.f; }
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        if (g_cnt > 0) {
            const uint32_t c0 = lds64(list_s + (uint32_t)g_begin * 8u).y >> KVR_CL_C0_SHIFT;
            fetch_half(ringK, g0K, c0, 0u);
            fetch_half(ringV, g0V, c0, 0u);
        }
        for (int base = 0; base < half; base += TPH) {           // TPH tokens per group and tile
            unsigned live = 0u;
#pragma unroll
            for (int h = 0; h < 2 * MT; ++h) {
                const int cnt_h = min(half, w1 - w0 - min(h * half, w1 - w0));
#pragma unroll
                for (int it = 0; it < TPH; ++it)
                    if (base + it < cnt_h) live |= 1u << (8 * (h >> 1) + 2 * it + (h & 1));
            }
            // ---- keys of the tile (Algorithm 2 on the key halves)
#pragma unroll 1
            for (int it = 0; it < TPH; ++it) {
                const bool lv = base + it < g_cnt;
                const uint2 e = lds64(list_s + (uint32_t)(lv ? g_begin + base + it : 0) * 8u);
                if (lv && ((e.y & KVR_CL_FLAG) || base + it == 0)) switch_run(k0, ringK, g0K, e.x >> KVR_CL_NEXT_SHIFT);
                const uint32_t a1 = lane_cells + (e.x & 0xFFu) * MQ_CELLB, a2 = lane_cells + ((e.x >> 8) & 0xFFu) * MQ_CELLB;
                const uint32_t dst = (uint32_t)((8 * wt + 2 * it + gw) * MQ_PITCH + lg * 8);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float4 kb = lds128(a1 + c * 256), kc = lds128(a2 + c * 256);
                    const float m0 = kvr_med3(k0[4 * c], kb.x, kc.x), m1 = kvr_med3(k0[4 * c + 1], kb.y, kc.y);
                    const float m2 = kvr_med3(k0[4 * c + 2], kb.z, kc.z), m3 = kvr_med3(k0[4 * c + 3], kb.w, kc.w);
                    uint32_t h0, h1, l0, l1;
                    split2(m0, m1, h0, l0);
                    split2(m2, m3, h1, l1);
                    sts64(tile_hi + dst + c * 128, h0, h1);
                    sts64(tile_lo + dst + c * 128, l0, l1);
                }
            }
            team_sync();
            qk_softmax(true, live, -1);
            team_sync();
            // ---- values of the tile; g_0 is applied to the median (med(g0 a, g1 b, g2 c) = g0 med(a, g0 g1 b, g0 g2 c))
#pragma unroll 1
            for (int it = 0; it < TPH; ++it) {
                const bool lv = base + it < g_cnt;
                const uint2 e = lds64(list_s + (uint32_t)(lv ? g_begin + base + it : 0) * 8u);
                if (lv && ((e.y & KVR_CL_FLAG) || base + it == 0)) switch_run(v0, ringV, g0V, e.x >> KVR_CL_NEXT_SHIFT);
                const uint32_t a1 = lane_cells + (e.x & 0xFFu) * MQ_CELLB + MQ_HALFB, a2 = lane_cells + ((e.x >> 8) & 0xFFu) * MQ_CELLB + MQ_HALFB;
                const float s0 = (e.y & (1u << KVR_CL_SIGN_SHIFT)) ? -1.f : 1.f;
                const float s01 = (e.y & (2u << KVR_CL_SIGN_SHIFT)) ? -1.f : 1.f, s02 = (e.y & (4u << KVR_CL_SIGN_SHIFT)) ? -1.f : 1.f;
                const uint32_t dst = (uint32_t)((8 * wt + 2 * it + gw) * MQ_PITCH + lg * 8);
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    const float4 vb = lds128(a1 + c * 256), vc = lds128(a2 + c * 256);
                    const float m0 = s0 * kvr_med3(v0[4 * c], s01 * vb.x, s02 * vc.x), m1 = s0 * kvr_med3(v0[4 * c + 1], s01 * vb.y, s02 * vc.y);
                    const float m2 = s0 * kvr_med3(v0[4 * c + 2], s01 * vb.z, s02 * vc.z), m3 = s0 * kvr_med3(v0[4 * c + 3], s01 * vb.w, s02 * vc.w);
                    uint32_t h0, h1, l0, l1;
                    split2(m0, m1, h0, l0);
                    split2(m2, m3, h1, l1);
                    sts64(tile_hi + dst + c * 128, h0, h1);
                    sts64(tile_lo + dst + c * 128, l0, l1);
                }
            }
            team_sync();
            pv(true);
            team_sync();
        }
    }
    asm volatile("cp.async.wait_all;\n" ::: "memory");

    // ---------------------------------------------------------------- the CTA's record: warps leave their
    // states where the cells were, one thread per (row, channel pair) folds them in warp order
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        l_run[h] += __shfl_xor_sync(FULL, l_run[h], 1);
        l_run[h] += __shfl_xor_sync(FULL, l_run[h], 2);
    }
    __syncthreads();                                        // every warp is done with the cells
    {
        float* scr = reinterpret_cast<float*>(smem + L.cells) + (size_t)warp * MQ_ROWS * PART;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) {
            *reinterpret_cast<float2*>(scr + fg * PART + 8 * nt + 2 * ft) = make_float2(O[nt][0], O[nt][1]);
            *reinterpret_cast<float2*>(scr + (fg + 8) * PART + 8 * nt + 2 * ft) = make_float2(O[nt][2], O[nt][3]);
        }
        if (ft == 0) {
            scr[fg * PART + KVR_D] = m_run[0]; scr[fg * PART + KVR_D + 1] = l_run[0];
            scr[(fg + 8) * PART + KVR_D] = m_run[1]; scr[(fg + 8) * PART + KVR_D + 1] = l_run[1];
        }
    }
    __syncthreads();
    {
        const float* scr = reinterpret_cast<const float*>(smem + L.cells);
        float* part = p.part + ((size_t)u * n_rec + rec) * ROWS_L * PART;
        for (int idx = tid; idx < ROWS_L * KVR_D; idx += MQ_THREADS) {
            const int rl = idx >> 7, d = idx & (KVR_D - 1);
            const int mt = rl / MQ_ROWS, r = rl % MQ_ROWS;              // the teams' warps that hold these 16 rows: t * MT + mt
            float M = M_EMPTY;
#pragma unroll
            for (int t = 0; t < NTEAMS; ++t) M = fmaxf(M, scr[((t * MT + mt) * MQ_ROWS + r) * PART + KVR_D]);
            float Ls = 0.f, Os = 0.f;
#pragma unroll
            for (int t = 0; t < NTEAMS; ++t) {
                const float f = ex2(scr[((t * MT + mt) * MQ_ROWS + r) * PART + KVR_D] - M);
                Ls += scr[((t * MT + mt) * MQ_ROWS + r) * PART + KVR_D + 1] * f;
                Os += scr[((t * MT + mt) * MQ_ROWS + r) * PART + d] * f;
            }
            part[rl * PART + d] = Os;
            if (d == 0) { part[rl * PART + KVR_D] = M; part[rl * PART + KVR_D + 1] = Ls; }
        }
    }
    // ---------------------------------------------------------------- last CTA of the head-instance merges
    __threadfence();
    __syncthreads();
    int* s_flag = reinterpret_cast<int*>(smem + L.ctrl);
    if (tid == 0) {
        const unsigned t = atomicAdd(&p.tickets[inst], 1u);
        *s_flag = (t == (unsigned)(n_rec - 1));
    }
    __syncthreads();
    if (!*s_flag) return;
    __threadfence();
    const float* recs = p.part + (size_t)u * n_rec * ROWS_L * PART;
    for (int idx = tid; idx < ROWS_L * KVR_D; idx += MQ_THREADS) {
        const int r = idx >> 7, d = idx & (KVR_D - 1);
        if (p.row0 + r >= p.M) continue;
        float M = M_EMPTY;
        for (int c = 0; c < n_rec; ++c) M = fmaxf(M, __ldcg(recs + ((size_t)c * ROWS_L + r) * PART + KVR_D));
        float Ls = 0.f, Os = 0.f;
        for (int c = 0; c < n_rec; ++c) {                  // fixed order: the result does not depend on timing
            const float* pr = recs + ((size_t)c * ROWS_L + r) * PART;
            const float f = ex2(__ldcg(pr + KVR_D) - M);
            Ls += __ldcg(pr + KVR_D + 1) * f;
            Os += __ldcg(pr + d) * f;
        }
        p.out[((size_t)u * p.M + p.row0 + r) * KVR_D + d] = Os / Ls;
    }
    if (tid == 0) p.tickets[inst] = 0u;
}

}  // namespace

// Records per head-instance and dynamic shared memory of the multi-query kernel, or false when the
// handle has no class grid (sketch too wide, or 8 query heads per kv head).
bool kvr_decode_mq_plan(const kvr_sketch* sk, int n_inst, int N, int R, int* S_out, int* lcap_out, size_t* smem_out) {
    const int C = sk->C, a = N - R;
    if (C < 1) return false;
    const int n_cls = C * C;
    int S = sk->n_sm / (n_inst * n_cls);
    if (S < 1) S = 1;
    const int s_cap = a / (n_cls * 4 * MQ_GROUPS) > 0 ? a / (n_cls * 4 * MQ_GROUPS) : 1;
    if (S > s_cap) S = s_cap;
    long long want = (long long)(a > 0 ? a : 1) / (n_cls * S);
    want += want / 8 + 64;
    const long long room = ((long long)MQ_SMEM_LIMIT - mq_layout(sk->n1, 0).total) / 8 - 4;
    if (room < 16) return false;
    if (want > room) want = room;
    want &= ~1LL;
    if (want < 2) want = 2;
    *S_out = S;
    *lcap_out = (int)want;
    *smem_out = (size_t)mq_layout(sk->n1, (int)want).total;
    return *smem_out <= MQ_SMEM_LIMIT;
}

size_t kvr_decode_mq_ws_bytes(int n_inst, int records) { return sizeof(float) * (size_t)n_inst * records * 4 * MQ_ROWS * kvr_dec::PART; }

cudaError_t kvr_launch_decode_mq(kvr_sketch* sk, int inst0, int n_inst, int rows, const void* q, const void* Kr, const void* Vr,
                                 int n_queries, int causal, float scale, float* out, int S, int lcap, size_t smem, float* part,
                                 cudaStream_t st) {
    MqParams p;
    p.q = q;
    p.Kr = (const uint2*)Kr;
    p.Vr = (const uint2*)Vr;
    p.cells = sk->cells;
    p.clist = sk->clist;
    p.coff = sk->coff;
    p.part = part;
    p.tickets = sk->tickets;
    p.out = out;
    p.status = sk->dev_status;
    p.inst0 = inst0;
    p.R = rows;
    p.b = sk->d.b;
    p.C = sk->C;
    p.logC = sk->logC;
    p.n1 = sk->n1;
    p.max_ctx = sk->d.max_context;
    p.S = S;
    p.lcap = lcap;
    p.M = sk->G * n_queries;
    p.Qn = n_queries;
    p.causal = causal;
    p.zero = 0u;
    p.scale_log2e = scale * 1.4426950408889634f;
    const bool f16 = sk->d.kv_dtype == KVR_F16;
    const dim3 grid(sk->C * sk->C * S, n_inst);
    // 64, 32 or 16 query rows per launch: as many as are left
    for (int row0 = 0; row0 < p.M;) {
        const int left = p.M - row0, mt = left > 32 ? 4 : left > 16 ? 2 : 1;
        void (*kern)(const MqParams) =
            mt == 4 ? (f16 ? decode_mq_kernel<__half, 4> : decode_mq_kernel<__nv_bfloat16, 4>)
          : mt == 2 ? (f16 ? decode_mq_kernel<__half, 2> : decode_mq_kernel<__nv_bfloat16, 2>)
                    : (f16 ? decode_mq_kernel<__half, 1> : decode_mq_kernel<__nv_bfloat16, 1>);
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        p.row0 = row0;
        kern<<<grid, MQ_THREADS, smem, st>>>(p);
        sk->launches += 1;
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        row0 += MQ_ROWS * mt;
    }
    return cudaSuccess;
}
