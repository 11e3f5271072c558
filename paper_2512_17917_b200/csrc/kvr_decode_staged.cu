// Decode attention over the mixed cache with the sketch cells staged in shared memory:
// Algorithm 4 (Revive) fused with p = Softmax(q K^T / sqrt(d_k)), out = p V of the Calculation
// Phase.
//
// A compressed token J needs the element-wise median of three cells (Algorithm 2),
//     K~_J[d] = med_i cellK[i][h_i(J)][d],     V~_J[d] = med_i g_i(J) cellV[i][h_i(J)][d],
// i.e. 3 KB of fp32 cell data fetched from three random places.  On-chip traffic, the min/max
// arithmetic of the medians and the instruction issue slots around them, not HBM bytes, are what this
// costs, so the kernel is organised around keeping cell reads on chip without any exchange between
// CTAs, and around keeping little state per lane so that many warps are resident:
//
//   * The compressed tokens of a head-instance are grouped into C x C classes by
//     (h_1(J) mod C, h_2(J) mod C).  All tokens of class (i, j) only touch the row-1 cells with
//     index = i (mod C) and the row-2 cells with index = j (mod C): 2 b / C cells of 1 KB (keys and
//     values, all 128 channels), which fit in one SM's shared memory.  One CTA stages that slice and
//     the class's token entries once (bulk copies that report to an mbarrier; the wait on it is
//     bounded) and serves the whole class, or a slice of it, from there.
//   * Inside a class the tokens are ordered by their row-0 cell.  The row-0 cell of the current run
//     of tokens stays in registers; the next run's cell (named by the entry that starts the run) is
//     fetched (cp.async) into the group's ring slot while the current run is processed.
//   * A group of 16 lanes takes one token at a time: each lane owns 8 channels (4 + 4, so that the
//     group reads 256 contiguous bytes of a cell per load, conflict-free).
//   * The work is done in two passes over the CTA's tokens (retained rows and compressed tokens alike):
//       key pass    a lane holds the scaled queries only; per token: medians of the key halves, the G
//                   partial dot products with packed two-wide fp32 FMAs, a select-free transposing
//                   shuffle tree (the lanes keep their queries in a head order permuted by lane, so
//                   every level sends a fixed half), the logit goes to shared memory;
//       weights     the CTA's maximum per head is known, so every logit becomes its softmax weight
//                   (sign g_0 of a reconstructed token folded in) in place, and the sum is formed;
//       value pass  a lane holds the output accumulators only; per token: medians of the value halves
//                   and G packed multiply-adds with the weights read back from shared memory.
//     Neither pass carries both the queries and the accumulators, there is no running maximum and no
//     rescaling inside the loops, and the groups of a CTA are merged by plain sums in a fixed order.
//   * Each CTA leaves one record (max, sum, o[G][128]); the last CTA of the head-instance to arrive
//     merges the records.  Nothing in this kernel waits on another CTA.
//   * SMs that the class grid leaves idle run CTAs that only stream retained rows.
#include <type_traits>

#include "kvr_decode_common.cuh"

namespace {
using namespace kvr_dec;
typedef unsigned long long u64;

constexpr int LPT = 16;             // lanes per token group: 8 channels per lane
constexpr int NT = 640;             // threads per CTA (at most 102 registers each)
constexpr int NGRP = NT / LPT;      // token groups per CTA
constexpr int NW = NT / 32;
constexpr int NC = 32 / LPT;        // 16-byte chunks (4 channels) per lane and vector
constexpr int NP = 2 * NC;          // packed pairs per lane and vector
constexpr int DPL = 4 * NC;         // channels per lane
constexpr int CELLF = 2 * KVR_D;    // floats of one staged cell: keys[128] | values[128]
constexpr int CELLB = CELLF * 4;
constexpr int HALFB = KVR_D * 4;    // bytes of the key half (or the value half) of a cell
constexpr unsigned FULL = 0xFFFFFFFFu;
constexpr size_t SMEM_LIMIT = 227 * 1024 - 2048;   // dynamic part; the kernel also has about 1.2 KB of static shared memory
// time of one retained row relative to one reconstructed token (measured): in a CTA that also serves
// a class and in a CTA that only streams rows
constexpr double COST_CLS = 0.45, COST_EXTRA = 0.45;

struct StagedParams {
    const void* q;          // [n_inst][G][128]  16-bit
    const uint2* Kr;        // [n_inst][R][32]   rows of 128 16-bit elements, as 8-byte pieces
    const uint2* Vr;
    const float* cells;     // handle base: [inst][2][r][b][128]
    const uint2* clist;     // handle base: [inst][max_ctx]
    const int32_t* coff;    // handle base: [inst][C*C+1]
    float* part;            // [n_inst][records][G][PART]
    uint32_t* tickets;      // handle base: [inst]
    float* out;             // [n_inst][G][128]
    int* status;            // handle's device status word: bit 0 set when a bounded wait gave up
    float* ml;              // handle base: [inst][G][2] reference maximum and sum of the softmax
    int inst0, R, b, C, logC, n1, max_ctx, S;
    int lcap;               // token entries staged at a time
    int rcap, rcap_extra;   // retained rows whose logits fit beside them (class CTAs / row-only CTAs)
    int n_ccta, r_cls;      // class CTAs per head-instance; retained rows they share (extra CTAs take the rest)
    float* emit;            // or null: [n_inst][emit_stride][G] every logit (log2 units): the rows, then the class-list entries
    int emit_stride;
    unsigned long long wait_ns;   // how long a wait on a staging barrier may last (200 ms unless a test shortens it)
    uint32_t tx_extra;      // 0; a test announces more bytes than are copied, so that the cells barrier never completes
    uint32_t zero;          // 0, unknown to the compiler (orders a shared-memory read before a copy into the same bytes)
    float scale_log2e;
};

__device__ __forceinline__ void cp_async16(uint32_t saddr, const void* gsrc) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(saddr), "l"(gsrc));
}
// 16 bytes of staged cell data at a 32-bit shared address + compile-time offset.  The staged cells
// do not change while tokens are processed, so these loads may be scheduled freely.
template <int OFF>
__device__ __forceinline__ float4 lds_cell(uint32_t addr) {
    float4 v;
    asm("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4+%5];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr), "n"(OFF));
    return v;
}
// compile-time loop (the loop index is needed as a constant for the load offsets)
template <int I, int N, typename F>
__device__ __forceinline__ void static_for(F&& f) {
    if constexpr (I < N) {
        f(std::integral_constant<int, I>{});
        static_for<I + 1, N>(f);
    }
}
// the same for memory that does change (ring slots, token entries, weights)
__device__ __forceinline__ float4 lds_vol(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];\n"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t lds_u32(uint32_t addr) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];\n" : "=r"(v) : "r"(addr) : "memory");
    return v;
}
__device__ __forceinline__ void sts_f32(uint32_t addr, float v) {
    asm volatile("st.shared.f32 [%0], %1;\n" ::"r"(addr), "f"(v) : "memory");
}
// ---- bulk copies global -> shared that report to an mbarrier ---------------------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(uint32_t sdst, const void* gsrc, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
                 ::"r"(sdst), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
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
// Bounded wait: the copies this kernel waits for take microseconds; a wait that lasts limit_ns
// gives up (the caller records it in the handle's status word) instead of hanging the GPU.
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
__device__ __forceinline__ uint2 ld_stream8(const uint2* p) {
    uint2 r;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p));
    return r;
}
// a load the compiler must leave where it stands (the queries are read again for every stretch of
// tokens instead of being kept in registers through the value pass)
__device__ __forceinline__ uint2 ld_here8(const uint2* p) {
    uint2 r;
    asm volatile("ld.global.v2.u32 {%0,%1}, [%2];" : "=r"(r.x), "=r"(r.y) : "l"(p) : "memory");
    return r;
}
// packed pairs of fp32 (sm_100 has two-wide fp32 multiply-add: half the issue slots)
__device__ __forceinline__ u64 pack2(float lo, float hi) {
    u64 r;
    asm("mov.b64 %0, {%1, %2};\n" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;\n" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c) {
    u64 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;\n" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ u64 add2(u64 a, u64 b) {
    u64 d;
    asm("add.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b) {
    u64 d;
    asm("mul.rn.f32x2 %0, %1, %2;\n" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
template <typename T>
__device__ __forceinline__ void unpack4(const uint2& x, u64 (&pr)[2]) {
    const float2 a = KvrType<T>::to_f2(x.x), b = KvrType<T>::to_f2(x.y);
    pr[0] = pack2(a.x, a.y);
    pr[1] = pack2(b.x, b.y);
}

// Shared-memory carve-up, in bytes from the start of the dynamic segment (all multiples of 16).
struct Layout {
    int ctrl, acc, ring, desc, stage, wbuf, cells, total;
};
// n1: cells per staged slice; lcap: token entries held at a time (even); rcap: retained rows whose
// logits are kept beside them; G: query heads per kv head
__host__ __device__ inline Layout make_layout(int n1, int lcap, int rcap, int G) {
    Layout L;
    int o = 0;
    L.ctrl = o;  o += 32;                            // last-arriver flag (int); at +16 and +24 the two staging mbarriers
    L.acc = o;   o += (G * PART * 4 + 15) & ~15;     // the CTA's record while stretches of tokens are folded into it
    L.ring = o;  o += NGRP * HALFB;                  // per token group: half of a row-0 cell in flight (also the merge scratch)
    L.desc = o;                                      // one 16-byte descriptor per token entry; the 8-byte entries
    L.stage = o + (lcap + 2) * 8;                    //   land in the upper half (+2: bulk copies move whole 16 bytes)
    o += (lcap + 2) * 16;
    L.wbuf = o;  o += ((rcap + lcap + 1) * G * 4 + 15) & ~15;   // one logit, later weight, per (token, head); + a zero slot
    L.cells = o; o += 2 * n1 * CELLB;                // row-1 slice, then row-2 slice
    L.total = o;
    return L;
}

// G: query heads per kv head.  MEAN: the three cells of a token are averaged instead of the paper's
// element-wise median (an option of the handle; the averages run on the two-wide fp32 multiply-add pipe).
template <typename T, int G, bool MEAN>
__global__ void __launch_bounds__(NT, 1)
decode_staged_kernel(const StagedParams p) {
    constexpr int LOGG = (G == 4) ? 2 : (G == 2) ? 1 : 0;
    constexpr int LGL = (LPT == 16) ? 4 : 3;
    constexpr int SH = LGL - LOGG;         // lanes (g << SH) .. of a group end up with head g's logit
    static_assert(LPT == 16 || LPT == 8, "lanes per token");
    static_assert(NT >= G * KVR_D && NT % 32 == 0 && NW <= 32, "one thread per (head, channel) folds the groups");
    extern __shared__ __align__(16) unsigned char smem[];
    // (g0 g1, g0 g1, g0 g2, g0 g2) for the 8 sign patterns of an entry; static shared memory sits at
    // the bottom of the window, so the table's address fits the 16 bits a descriptor has for it
    __shared__ __align__(128) float4 s_sign[8];
    __shared__ float s_red[32][4], s_redl[32][4];     // per warp and head: largest logit, sum of weights
    __shared__ float s_M[4], s_L[4];

    const Layout L = make_layout(p.n1, p.lcap, p.rcap, G);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, grp = tid / LPT, lg = tid & (LPT - 1);
    const int u = blockIdx.y, inst = p.inst0 + u, b = p.b, C = p.C, n1 = p.n1;
    const int rec = blockIdx.x, n_rec = gridDim.x;
    const bool extra = rec >= p.n_ccta;            // a CTA that only streams retained rows
    const int cls = extra ? 0 : rec / p.S, sp = rec - cls * p.S;
    const int ci = cls >> p.logC, cj = cls & (C - 1);
    if (tid < 8) s_sign[tid] = make_float4((tid & 2) ? -1.f : 1.f, (tid & 2) ? -1.f : 1.f, (tid & 4) ? -1.f : 1.f, (tid & 4) ? -1.f : 1.f);
    // A following decode launch may be scheduled as soon as every CTA of this one is running: its
    // CTAs take the SMs this launch frees one by one and stage their cells while this launch drains.
    asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");

    // (asked for first: the cell copies below do not need them, and they are back by the time they do)
    int k_lo = 0, k_hi = 0;
    if (!extra) {
        const int32_t* coff = p.coff + (size_t)inst * (C * C + 1);
        k_lo = __ldg(coff + cls);
        k_hi = __ldg(coff + cls + 1);
    }
    const uint32_t smem_s = (uint32_t)__cvta_generic_to_shared(smem);
    const uint32_t cells_s = smem_s + L.cells, desc_s = smem_s + L.desc, wbuf_s = smem_s + L.wbuf;
    // ---------------------------------------------------------------- start staging.  The class's cells
    // travel as bulk copies that report to one mbarrier, the first stretch of its token entries to a
    // second one.  The cell copies need nothing but the class number, so they go first; a warp issues
    // its copies one lane after the other, so they are dealt to the warps round-robin.
    const uint32_t bar_cells = smem_s + L.ctrl + 16u, bar_list = smem_s + L.ctrl + 24u;
    if (!extra) {
        const float* cellsK = p.cells + (size_t)inst * 2 * KVR_R * b * KVR_D;
        const float* cellsV = cellsK + (size_t)KVR_R * b * KVR_D;
        if (tid == 0) {
            mbar_init(bar_cells, 1);
            mbar_init(bar_list, 1);
            const int cnt1 = (b - ci + C - 1) >> p.logC, cnt2 = (b - cj + C - 1) >> p.logC;   // cells of the two slices
            mbar_expect_tx(bar_cells, (uint32_t)((cnt1 + cnt2) * CELLB) + p.tx_extra);
        }
        __syncthreads();
        for (int i = warp + lane * NW; i < 4 * n1; i += NT) {       // one 512-byte piece per (cell, keys | values)
            const int idx = i >> 1, kv = i & 1;
            const int h = (idx < n1) ? idx * C + ci : (idx - n1) * C + cj;
            const int row = (idx < n1) ? 1 : 2;
            if (h < b)
                bulk_g2s(cells_s + (uint32_t)(idx * CELLB + kv * HALFB),
                         (kv ? cellsV : cellsK) + ((size_t)row * b + h) * KVR_D, HALFB, bar_cells);
        }
    }
    // this CTA's slice of its class, and its retained rows
    int s_begin = 0, s_end = 0, r_begin, r_end;
    if (!extra) {
        const int k_len = k_hi - k_lo;
        s_begin = k_lo + (int)((long long)k_len * sp / p.S);
        s_end = k_lo + (int)((long long)k_len * (sp + 1) / p.S);
        r_begin = (int)((long long)p.r_cls * rec / p.n_ccta);
        r_end = (int)((long long)p.r_cls * (rec + 1) / p.n_ccta);
    } else {
        const int e = rec - p.n_ccta, n_e = n_rec - p.n_ccta, rest = p.R - p.r_cls;
        r_begin = p.r_cls + (int)((long long)rest * e / n_e);
        r_end = p.r_cls + (int)((long long)rest * (e + 1) / n_e);
    }
    const int lcap = p.lcap, rcap = extra ? p.rcap_extra : p.rcap;
    const uint2* clist = p.clist + (size_t)inst * p.max_ctx;
    const int len0 = min(lcap, s_end - s_begin);
    // a bulk copy starts on 16 bytes: take the entry before, if need be (entries are 8 bytes)
    const int lshift = (int)(((size_t)inst * p.max_ctx + s_begin) & 1);
    if (len0 > 0 && tid == 0) {
        const uint32_t bytes = (uint32_t)(((len0 + lshift + 1) & ~1) * 8);
        mbar_expect_tx(bar_list, bytes);
        bulk_g2s(smem_s + L.stage, clist + (s_begin - lshift), bytes, bar_list);
    }
    // The rows are read twice (keys, later values), microseconds apart: ask for all of them now, so
    // that both reads find them in the L2 cache instead of waiting for HBM one batch at a time.  A
    // request occupies its warp until the copy engine has taken it (about a microsecond per 8 KB
    // when megabytes are asked for), so a CTA with many rows leaves all of them to its last warp,
    // keys first, while the other warps start on the rows that have arrived.
    {
        constexpr int PF = 8192;                            // bytes per prefetch request (32 rows)
        const char* k8 = reinterpret_cast<const char*>(p.Kr + ((size_t)u * p.R + r_begin) * 32);
        const char* v8 = reinterpret_cast<const char*>(p.Vr + ((size_t)u * p.R + r_begin) * 32);
        const int bytes = (r_end - r_begin) * 256;
        if (bytes <= NW * PF) {
            for (int o = (warp + lane * NW) * PF; o < bytes; o += NT * PF) {     // (dealt to the warps like the cell copies)
                const uint32_t n = (uint32_t)min(PF, bytes - o);
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(k8 + o), "r"(n) : "memory");
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(v8 + o), "r"(n) : "memory");
            }
        } else if (warp == NW - 1) {
            for (int o = lane * PF; o < bytes; o += 32 * PF)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(k8 + o), "r"((uint32_t)min(PF, bytes - o)) : "memory");
            for (int o = lane * PF; o < bytes; o += 32 * PF)
                asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;\n" ::"l"(v8 + o), "r"((uint32_t)min(PF, bytes - o)) : "memory");
        }
    }
    // stretches: the tokens are taken lcap entries and rcap rows at a time (normally all at once)
    int n_str = 1;
    {
        const int a_ = (s_end - s_begin + lcap - 1) / lcap, b_ = (r_end - r_begin + rcap - 1) / rcap;
        n_str = max(1, max(a_, b_));
    }
    const uint32_t wzero_s = wbuf_s + (uint32_t)(extra ? p.rcap_extra : p.rcap + lcap) * (G * 4);
    const uint32_t sign_s = (uint32_t)__cvta_generic_to_shared(s_sign);
    float* s_acc = reinterpret_cast<float*>(smem + L.acc);
    // Row-0 cells: each lane moves its own 16-byte pieces of the key half or the value half of a cell
    // into its group's ring slot, and later reads exactly those bytes back.  g0 = this lane's piece of
    // that half of row-0 cell 0.
    const uint32_t ring_s = smem_s + L.ring + (uint32_t)(grp * HALFB + lg * 16);
    auto fetch_row0 = [&](const float* g0, uint32_t c0, uint32_t z) {
        const float* g = g0 + (size_t)c0 * KVR_D;
#pragma unroll
        for (int c = 0; c < NC; ++c) cp_async16(ring_s + z + c * LPT * 16, g + c * LPT * 4);
        asm volatile("cp.async.commit_group;\n" ::);
    };
    // Take the fetched half cell into registers and ask for the next run's.  The copy must not start
    // before the bytes are read: its address is made to depend on the loaded values (z is always 0).
    auto switch_run = [&](float (&r0v)[DPL], const float* g0, uint32_t c0_next) {
        asm volatile("cp.async.wait_all;\n" ::: "memory");
        uint32_t z = 0;
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const float4 a = lds_vol(ring_s + c * LPT * 16);
            r0v[4 * c] = a.x; r0v[4 * c + 1] = a.y; r0v[4 * c + 2] = a.z; r0v[4 * c + 3] = a.w;
            z |= __float_as_uint(a.w);
        }
        fetch_row0(g0, c0_next, z & p.zero);
    };
    // the group's share of a stretch of `len` entries: the first rn groups take qn + 1 tokens, the others qn
    auto share = [&](int len, int& qn, int& rn, int& r0) {
        qn = len / NGRP;
        rn = len - qn * NGRP;
        r0 = grp * qn + min(grp, rn);
    };
    uint32_t c0_first = 0;                                     // row-0 cell of the group's first token
    const int own = lg >> SH;                                  // the head whose logit this lane ends up with
    const uint32_t lane16 = (uint32_t)(lg * 16);

    for (int st = 0; st < n_str; ++st) {
        const int rb = min(r_begin + st * rcap, r_end), re = min(rb + rcap, r_end), nrows = re - rb;
        const int cb = min(s_begin + st * lcap, s_end), len = min(lcap, s_end - cb);
        int qn, rn, r0;
        share(len, qn, rn, r0);
        const bool ragged_live = grp < rn;                     // this group has a token in the ragged last round
        if (st > 0) {
            __syncthreads();                                   // previous stretch consumed
            asm volatile("cp.async.wait_all;\n" ::: "memory");
        }
        // ------------------------------------------------------------ key pass
        // The scaled queries, head order permuted by lane: slot i holds head i ^ own, so that every
        // level of the shuffle tree below keeps its low slots and sends its high slots.
        u64 q2[G][NP];
        {
            const uint2* qg = reinterpret_cast<const uint2*>(p.q) + (size_t)u * G * 32;     // 32 8-byte pieces per head
            const u64 sc2 = pack2(p.scale_log2e, p.scale_log2e);
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    u64 t2[2];
                    unpack4<T>(ld_here8(qg + (g ^ own) * 32 + c * LPT + lg), t2);
                    q2[g][2 * c] = mul2(t2[0], sc2);
                    q2[g][2 * c + 1] = mul2(t2[1], sc2);
                }
            }
        }
        // logit (log2 units) of head `own` for the token whose key channels are kp
        auto logit = [&](const u64 (&kp)[NP]) -> float {
            float s[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                u64 acc = mul2(q2[g][0], kp[0]);
#pragma unroll
                for (int k = 1; k < NP; ++k) acc = fma2(q2[g][k], kp[k], acc);
                float lo, hi;
                unpack2(acc, lo, hi);
                s[g] = lo + hi;
            }
            float mine;
            if constexpr (G == 4) {
                const float t0 = s[0] + __shfl_xor_sync(FULL, s[2], LPT / 2);
                const float t1 = s[1] + __shfl_xor_sync(FULL, s[3], LPT / 2);
                mine = t0 + __shfl_xor_sync(FULL, t1, LPT / 4);
#pragma unroll
                for (int x = LPT / 8; x >= 1; x >>= 1) mine += __shfl_xor_sync(FULL, mine, x);
            } else if constexpr (G == 2) {
                mine = s[0] + __shfl_xor_sync(FULL, s[1], LPT / 2);
#pragma unroll
                for (int x = LPT / 4; x >= 1; x >>= 1) mine += __shfl_xor_sync(FULL, mine, x);
            } else {
                mine = s[0];
#pragma unroll
                for (int x = LPT / 2; x >= 1; x >>= 1) mine += __shfl_xor_sync(FULL, mine, x);
            }
            return mine;
        };
        float mx = M_EMPTY;                                        // largest logit this lane has seen (head `own`)
        constexpr int FLB = (LPT == 16) ? 8 : 4, FLT = (LPT == 16) ? 2 : 1;                            // rows per group in flight: full blocks, tail
        // retained rows (exact keys): row t of the stretch goes to group t mod NGRP.  All lanes of a
        // (token, head) quad hold the same logit and store it to the same word.
        if (nrows > 0) {
            const uint2* Kr = p.Kr + ((size_t)u * p.R + rb) * 32 + lg;
            const uint32_t wb0 = wbuf_s + (uint32_t)(own * 4);
            auto rows_key = [&](auto FLc, auto CHK, int base) {
                constexpr int FLn = decltype(FLc)::value;
                constexpr bool CHECK = decltype(CHK)::value;
                const uint2* kb = Kr + (size_t)(base + grp) * 32;
                uint2 kx[FLn][NC];
#pragma unroll
                for (int i = 0; i < FLn; ++i) {
                    const bool ok = !CHECK || base + i * NGRP + grp < nrows;
#pragma unroll
                    for (int c = 0; c < NC; ++c) kx[i][c] = ld_stream8((ok ? kb + i * NGRP * 32 : Kr) + c * LPT);
                }
                const uint32_t wb = wb0 + (uint32_t)(base + grp) * (G * 4);
#pragma unroll
                for (int i = 0; i < FLn; ++i) {
                    u64 kp[NP], t2[2];
#pragma unroll
                    for (int c = 0; c < NC; ++c) { unpack4<T>(kx[i][c], t2); kp[2 * c] = t2[0]; kp[2 * c + 1] = t2[1]; }
                    const float mine = logit(kp);
                    if (!CHECK || base + i * NGRP + grp < nrows) {
                        mx = fmaxf(mx, mine);
                        sts_f32(wb + i * NGRP * G * 4, mine);
                    }
                }
            };
            int base = 0;
            for (; base + FLB * NGRP <= nrows; base += FLB * NGRP) rows_key(std::integral_constant<int, FLB>{}, std::false_type{}, base);
            for (; base < nrows; base += FLT * NGRP) rows_key(std::integral_constant<int, FLT>{}, std::true_type{}, base);
        }
        // ------------------------------------------------------------ token entries -> descriptors
        // One thread per entry turns the 8-byte entry into what the two token loops need without further
        // arithmetic: x, y = shared addresses of its row-1 and row-2 cells, z = address of its logit /
        // weight slot, w = row-0 cell of the next run << 16 | address of its sign pairs | run flag
        // (also set for the first token of every group).  The entries lie in the upper half of the
        // descriptor array; a batch of descriptors only overwrites entries that were read before.
        if (st == 0 && len0 > 0 && !mbar_wait(bar_list, 0, p.wait_ns)) atomicOr(p.status, 1);       // the first entries have landed
        const float* g0K = p.cells + (size_t)inst * 2 * KVR_R * b * KVR_D + 4 * lg;      // this lane's piece of row-0 cell 0, key half
        {
            const uint2* staged = reinterpret_cast<const uint2*>(smem + L.stage) + lshift;
            uint4* desc = reinterpret_cast<uint4*>(smem + L.desc);
            // each group asks for the row-0 key half of its first token
            if (qn + (ragged_live ? 1 : 0) > 0) {
                c0_first = ((st == 0) ? staged[r0].y : __ldg(&clist[cb + r0].y)) >> KVR_CL_C0_SHIFT;
                fetch_row0(g0K, c0_first, 0u);
            }
            const int split = rn * (qn + 1);
            constexpr int EPT = 4;                             // entries a thread holds at a time
            for (int base = 0; base < len; base += EPT * NT) {
                uint2 e[EPT];
#pragma unroll
                for (int k = 0; k < EPT; ++k) {
                    const int i = base + k * NT + tid;
                    e[k] = make_uint2(0u, 0u);
                    if (i < len) e[k] = (st == 0) ? staged[i] : clist[cb + i];
                }
                __syncthreads();
#pragma unroll
                for (int k = 0; k < EPT; ++k) {
                    const int i = base + k * NT + tid;
                    if (i < len) {
                        bool start = true;                     // first token of its group?
                        if (qn > 0) start = (i < split) ? (i % (qn + 1) == 0) : ((i - split) % qn == 0);
                        uint4 d;
                        d.x = cells_s + (e[k].x & 0xFFu) * CELLB;
                        d.y = cells_s + ((e[k].x >> 8) & 0xFFu) * CELLB;
                        d.z = wbuf_s + (uint32_t)(nrows + i) * (G * 4);
                        d.w = (e[k].x & 0xFFFF0000u) | (sign_s + (e[k].y & 0x70u)) | (e[k].y & KVR_CL_FLAG) | (start ? KVR_CL_FLAG : 0u);
                        desc[i] = d;
                    }
                }
            }
            __syncthreads();
        }
        if (st == 0 && !extra && !mbar_wait(bar_cells, 0, p.wait_ns)) atomicOr(p.status, 1);       // the cells have landed
        // compressed tokens (Algorithm 2 on the key halves)
        if (len > 0) {
            float k0[DPL];                                // key half of the run's row-0 cell (this lane's channels)
#pragma unroll
            for (int x = 0; x < DPL; ++x) k0[x] = 0.f;
            const uint32_t own4 = (uint32_t)(own * 4);
            auto key_token = [&](uint32_t dp, bool live) {
                uint4 d;
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(d.x), "=r"(d.y), "=r"(d.z), "=r"(d.w) : "r"(dp) : "memory");
                if (live && (d.w & KVR_CL_FLAG)) switch_run(k0, g0K, d.w >> KVR_CL_NEXT_SHIFT);
                const uint32_t a1 = d.x + lane16, a2 = d.y + lane16;
                u64 kp[NP];
                static_for<0, NC>([&](auto ic) {
                    constexpr int c = decltype(ic)::value;
                    const float4 kb = lds_cell<c * LPT * 16>(a1), kc = lds_cell<c * LPT * 16>(a2);
                    if constexpr (MEAN) {
                        const u64 third2 = pack2(1.0f / 3.0f, 1.0f / 3.0f);
                        kp[2 * c] = mul2(add2(pack2(kc.x, kc.y), add2(pack2(kb.x, kb.y), pack2(k0[4 * c], k0[4 * c + 1]))), third2);
                        kp[2 * c + 1] = mul2(add2(pack2(kc.z, kc.w), add2(pack2(kb.z, kb.w), pack2(k0[4 * c + 2], k0[4 * c + 3]))), third2);
                    } else {
                        kp[2 * c] = pack2(kvr_med3(k0[4 * c], kb.x, kc.x), kvr_med3(k0[4 * c + 1], kb.y, kc.y));
                        kp[2 * c + 1] = pack2(kvr_med3(k0[4 * c + 2], kb.z, kc.z), kvr_med3(k0[4 * c + 3], kb.w, kc.w));
                    }
                });
                const float mine = logit(kp);
                if (live) {
                    mx = fmaxf(mx, mine);
                    sts_f32(d.z + own4, mine);
                }
            };
            uint32_t dp = desc_s + (uint32_t)r0 * 16u;
#pragma unroll 1
            for (int it = 0; it < qn; ++it, dp += 16) key_token(dp, true);
            if (rn > 0) key_token(ragged_live ? dp : desc_s, ragged_live);      // ragged last round
            // the value half of the first token's row-0 cell, for the value pass
            asm volatile("cp.async.wait_all;\n" ::: "memory");
            if (qn + (ragged_live ? 1 : 0) > 0) fetch_row0(g0K + (size_t)KVR_R * b * KVR_D, c0_first, 0u);
        }
        // the warp's largest logits per head (the lanes of a (token, head) quad hold the same value)
#pragma unroll
        for (int x = LPT; x < 32; x <<= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, x));
        if (lane < LPT && (lg & ((1 << SH) - 1)) == 0) s_red[warp][own] = mx;
        __syncthreads();
        // ------------------------------------------------------------ logits -> weights, in place: the
        // CTA's maximum per head (every warp folds the warps' maxima itself), then
        // w = 2^(logit - max) (times g_0 for a reconstructed token), and the warps' sums
        {
            const int n_tok = nrows + len;
            float* w = reinterpret_cast<float*>(smem + L.wbuf);
            float M[G], l[G];
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float v = lane < NW ? s_red[lane][g] : M_EMPTY;
#pragma unroll
                for (int x = 1; x < 32; x <<= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, x));
                M[g] = v;
                l[g] = 0.f;
            }
            if (tid < G) {
                float m = M[0];
#pragma unroll
                for (int g = 1; g < G; ++g) m = (tid == g) ? M[g] : m;
                s_M[tid] = m;
            }
            for (int t = tid; t < n_tok; t += NT) {
                float x[G];
                if constexpr (G == 4) { const float4 v = *reinterpret_cast<const float4*>(w + 4 * t); x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
                else if constexpr (G == 2) { const float2 v = *reinterpret_cast<const float2*>(w + 2 * t); x[0] = v.x; x[1] = v.y; }
                else x[0] = w[t];
                if (p.emit) {                                // (same for the whole launch)
                    float* e = p.emit + ((size_t)u * p.emit_stride + (t < nrows ? rb + t : p.R + cb + (t - nrows))) * G;
                    if constexpr (G == 4) *reinterpret_cast<float4*>(e) = make_float4(x[0], x[1], x[2], x[3]);
                    else if constexpr (G == 2) *reinterpret_cast<float2*>(e) = make_float2(x[0], x[1]);
                    else e[0] = x[0];
                }
                float sgn = 1.f;
                if (t >= nrows) {
                    if (lds_u32(desc_s + (uint32_t)(t - nrows) * 16u + 12u) & (1u << KVR_CL_SIGN_SHIFT)) sgn = -1.f;   // g_0
                    if (MEAN) sgn *= (1.0f / 3.0f);
                }
#pragma unroll
                for (int g = 0; g < G; ++g) {
                    const float pr = ex2(x[g] - M[g]);
                    l[g] += pr;
                    x[g] = pr * sgn;
                }
                if constexpr (G == 4) *reinterpret_cast<float4*>(w + 4 * t) = make_float4(x[0], x[1], x[2], x[3]);
                else if constexpr (G == 2) *reinterpret_cast<float2*>(w + 2 * t) = make_float2(x[0], x[1]);
                else w[t] = x[0];
            }
            if (tid < G) w[(extra ? p.rcap_extra : p.rcap + lcap) * G + tid] = 0.f;    // the weight of a filler token
#pragma unroll
            for (int g = 0; g < G; ++g) {
#pragma unroll
                for (int x = 1; x < 32; x <<= 1) l[g] += __shfl_xor_sync(FULL, l[g], x);   // a fixed tree: same sum every run
                if (lane == 0) s_redl[warp][g] = l[g];
            }
            __syncthreads();
        }
        // ------------------------------------------------------------ value pass
        u64 o2[G][NP];
#pragma unroll
        for (int g = 0; g < G; ++g)
#pragma unroll
            for (int k = 0; k < NP; ++k) o2[g][k] = 0ull;
        // o[g] += w[g] * v for the token whose weights sit at shared address wa
        auto add_token = [&](uint32_t wa, const u64 (&vp)[NP]) {
            float wg[G];
            if constexpr (G == 4) {
                const float4 w4 = lds_vol(wa);
                wg[0] = w4.x; wg[1] = w4.y; wg[2] = w4.z; wg[3] = w4.w;
            } else if constexpr (G == 2) {
                asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];\n" : "=f"(wg[0]), "=f"(wg[1]) : "r"(wa) : "memory");
            } else {
                asm volatile("ld.shared.f32 %0, [%1];\n" : "=f"(wg[0]) : "r"(wa) : "memory");
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const u64 w2 = pack2(wg[g], wg[g]);
#pragma unroll
                for (int k = 0; k < NP; ++k) o2[g][k] = fma2(w2, vp[k], o2[g][k]);
            }
        };
        if (nrows > 0) {
            const uint2* Vr = p.Vr + ((size_t)u * p.R + rb) * 32 + lg;
            auto rows_val = [&](auto FLc, auto CHK, int base) {
                constexpr int FLn = decltype(FLc)::value;
                constexpr bool CHECK = decltype(CHK)::value;
                const uint2* vb = Vr + (size_t)(base + grp) * 32;
                uint2 vx[FLn][NC];
#pragma unroll
                for (int i = 0; i < FLn; ++i) {
                    const bool ok = !CHECK || base + i * NGRP + grp < nrows;
#pragma unroll
                    for (int c = 0; c < NC; ++c) vx[i][c] = ld_stream8((ok ? vb + i * NGRP * 32 : Vr) + c * LPT);
                }
                const uint32_t wa = wbuf_s + (uint32_t)(base + grp) * (G * 4);
#pragma unroll
                for (int i = 0; i < FLn; ++i) {
                    u64 vp[NP], t2[2];
#pragma unroll
                    for (int c = 0; c < NC; ++c) { unpack4<T>(vx[i][c], t2); vp[2 * c] = t2[0]; vp[2 * c + 1] = t2[1]; }
                    add_token((!CHECK || base + i * NGRP + grp < nrows) ? wa + i * NGRP * G * 4 : wzero_s, vp);
                }
            };
            int base = 0;
            for (; base + FLB * NGRP <= nrows; base += FLB * NGRP) rows_val(std::integral_constant<int, FLB>{}, std::false_type{}, base);
            for (; base < nrows; base += FLT * NGRP) rows_val(std::integral_constant<int, FLT>{}, std::true_type{}, base);
        }
        if (len > 0) {
            float v0[DPL];
#pragma unroll
            for (int x = 0; x < DPL; ++x) v0[x] = 0.f;
            const float* g0V = g0K + (size_t)KVR_R * b * KVR_D;
            auto val_token = [&](uint32_t dp, bool live) {
                uint4 d;
                asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n" : "=r"(d.x), "=r"(d.y), "=r"(d.z), "=r"(d.w) : "r"(dp) : "memory");
                if (live && (d.w & KVR_CL_FLAG)) switch_run(v0, g0V, d.w >> KVR_CL_NEXT_SHIFT);
                const uint32_t a1 = d.x + lane16, a2 = d.y + lane16;
                // med(g0 a, g1 b, g2 c) = g0 med(a, g0 g1 b, g0 g2 c): g0 is part of the weight
                const float4 sg = lds_vol(d.w & 0xFFF0u);
                const u64 g01p = pack2(sg.x, sg.y), g02p = pack2(sg.z, sg.w);
                u64 vp[NP];
                static_for<0, NC>([&](auto ic) {
                    constexpr int c = decltype(ic)::value;
                    const float4 vb = lds_cell<HALFB + c * LPT * 16>(a1), vc = lds_cell<HALFB + c * LPT * 16>(a2);
                    if constexpr (MEAN) {
                        // (the sum of the three; its third is part of the weight)
                        vp[2 * c] = fma2(pack2(vc.x, vc.y), g02p, fma2(pack2(vb.x, vb.y), g01p, pack2(v0[4 * c], v0[4 * c + 1])));
                        vp[2 * c + 1] = fma2(pack2(vc.z, vc.w), g02p, fma2(pack2(vb.z, vb.w), g01p, pack2(v0[4 * c + 2], v0[4 * c + 3])));
                        return;
                    }
                    float b0, b1, b2, b3, c0, c1, c2, c3;
                    unpack2(mul2(pack2(vb.x, vb.y), g01p), b0, b1);
                    unpack2(mul2(pack2(vb.z, vb.w), g01p), b2, b3);
                    unpack2(mul2(pack2(vc.x, vc.y), g02p), c0, c1);
                    unpack2(mul2(pack2(vc.z, vc.w), g02p), c2, c3);
                    vp[2 * c] = pack2(kvr_med3(v0[4 * c], b0, c0), kvr_med3(v0[4 * c + 1], b1, c1));
                    vp[2 * c + 1] = pack2(kvr_med3(v0[4 * c + 2], b2, c2), kvr_med3(v0[4 * c + 3], b3, c3));
                });
                add_token(live ? d.z : wzero_s, vp);
            };
            uint32_t dp = desc_s + (uint32_t)r0 * 16u;
#pragma unroll 1
            for (int it = 0; it < qn; ++it, dp += 16) val_token(dp, true);
            if (rn > 0) val_token(ragged_live ? dp : desc_s, ragged_live);
        }
        // ------------------------------------------------------------ add up the groups of this CTA (they
        // share one maximum, so this is a plain sum in a fixed order) and fold the stretch into the record
        asm volatile("cp.async.wait_all;\n" ::: "memory");         // no copy into the ring is in flight
        {
            // every group leaves its sums in shared memory, as many groups at a time as fit between
            // the ring and the cells (descriptors and weights are no longer needed); one thread per
            // (head, channel) adds them in group order
            float* scr = reinterpret_cast<float*>(smem + L.ring);   // [groups at a time][G][128]
            const int fit = min(NGRP, (L.cells - L.ring) / (G * HALFB));
            float sum = 0.f;
            for (int g0 = 0; g0 < NGRP; g0 += fit) {
                __syncthreads();
                if (grp >= g0 && grp < g0 + fit) {
                    float* r = scr + (size_t)(grp - g0) * G * KVR_D;
#pragma unroll
                    for (int g = 0; g < G; ++g)
#pragma unroll
                        for (int c = 0; c < NC; ++c) {
                            float4 v;
                            unpack2(o2[g][2 * c], v.x, v.y);
                            unpack2(o2[g][2 * c + 1], v.z, v.w);
                            *reinterpret_cast<float4*>(r + g * KVR_D + (c * LPT + lg) * 4) = v;
                        }
                }
                if (g0 == 0 && warp == 0) {                  // the CTA's sums of weights (fixed tree)
#pragma unroll
                    for (int g = 0; g < G; ++g) {
                        float v = lane < NW ? s_redl[lane][g] : 0.f;
#pragma unroll
                        for (int x = 1; x < 32; x <<= 1) v += __shfl_xor_sync(FULL, v, x);
                        if (lane == 0) s_L[g] = v;
                    }
                }
                __syncthreads();
                if (tid < G * KVR_D) {
                    const int n = min(fit, NGRP - g0);
#pragma unroll 4
                    for (int w = 0; w < n; ++w) sum += scr[w * G * KVR_D + tid];
                }
            }
            const int g = tid >> 7, d = tid & (KVR_D - 1);
            float Mo = M_EMPTY, Lo = 0.f, Oo = 0.f;
            if (st > 0 && tid < G * KVR_D) { Mo = s_acc[g * PART + KVR_D]; Lo = s_acc[g * PART + KVR_D + 1]; Oo = s_acc[g * PART + d]; }
            if (st > 0) __syncthreads();
            if (tid < G * KVR_D) {
                const float Ms = s_M[g], Mn = fmaxf(Mo, Ms);
                const float f0 = ex2(Mo - Mn), f1 = ex2(Ms - Mn);
                s_acc[g * PART + d] = Oo * f0 + sum * f1;
                if (d == 0) { s_acc[g * PART + KVR_D] = Mn; s_acc[g * PART + KVR_D + 1] = Lo * f0 + s_L[g] * f1; }
            }
        }
    }
    // ---------------------------------------------------------------- everything above reads only what no
    // decode launch writes (cells, token lists, the caller's rows and queries) and writes shared
    // memory only.  When this launch was made a programmatic dependent of the previous decode launch,
    // its CTAs took over the SMs that launch freed one by one and may have run beside its last CTAs:
    // wait for that launch to be complete here, before the first write to global memory (records,
    // tickets, outputs are shared by consecutive launches).
    asm volatile("griddepcontrol.wait;\n" ::: "memory");
    __syncthreads();
    {
        float* part = p.part + ((size_t)blockIdx.y * gridDim.x + blockIdx.x) * G * PART;
        for (int i = tid; i < G * PART; i += NT) part[i] = s_acc[i];
    }
    finish_instance<G, NT>(p.part + (size_t)blockIdx.y * gridDim.x * G * PART, (int)gridDim.x, &p.tickets[p.inst0 + blockIdx.y],
                           p.out + (size_t)blockIdx.y * G * KVR_D, p.ml + (size_t)(p.inst0 + blockIdx.y) * G * 2,
                           reinterpret_cast<int*>(smem + L.ctrl));
}

// chained: the previous kernel of the stream is a staged decode launch of the same handle and nothing
// has changed the handle's cells or lists since, so this launch may overlap its start with that
// launch's end (programmatic dependent launch; the kernel waits before it touches anything shared).
template <typename T, int G, bool MEAN>
cudaError_t launch_one(const StagedParams& p, int n_inst, int grid_x, size_t smem, bool chained, cudaStream_t st) {
    auto kern = decode_staged_kernel<T, G, MEAN>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid_x, n_inst);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, p);
}

}  // namespace

// Smallest class grid whose rows-1-and-2 slices leave room for the ring and a useful number of
// token entries and logits; 0 when the sketch is too wide (or the query group too large) for this kernel.
int kvr_decode_staged_pick_C(int b, int G) {
    if (G != 1 && G != 2 && G != 4) return 0;
    for (int C = 1; C <= 8; C *= 2) {
        const int n1 = (b + C - 1) / C;
        if (2 * n1 <= 226 && (size_t)make_layout(n1, 1536, 768, G).total <= SMEM_LIMIT) return C;
    }
    return 0;
}

// How the staged kernel would run this call, or `false` when it cannot (no class grid fits) or
// should not (so few tokens that almost every one would fetch its own row-0 cell from global memory).
bool kvr_decode_staged_plan(const kvr_sketch* sk, int n_inst, int N, int R, int rows, bool forced,
                            KvrStagedPlan* plan) {
    const int a = N - R, C = sk->C, G = sk->G;
    R = rows;                                   // from here on: the rows to stream
    if (C < 1 || a < 1) return false;
    const int n_cls = C * C;
    if (!forced && 2LL * a < (long long)sk->d.b * n_cls) return false;   // under half a token per (class, row-0 cell)
    int S = sk->n_sm / (n_inst * n_cls);                      // one CTA per SM
    if (S < 1) S = 1;
    const int s_cap = a / (n_cls * 2 * NGRP) > 0 ? a / (n_cls * 2 * NGRP) : 1;   // a couple of tokens per group at least
    if (S > s_cap) S = s_cap;
    // SMs the class CTAs leave idle stream retained rows only.  The rows are dealt so that all CTAs
    // finish at about the same time.
    const int n_ccta = n_cls * S;
    int extra = (sk->n_sm - n_inst * n_ccta) / n_inst;
    if (extra < 0 || R < 1) extra = 0;
    if (extra > 8) extra = 8;
    int r_cls = R;
    if (extra > 0) {
        // x rows per class CTA, y per extra CTA:  n_ccta x + extra y = R,  tokens + COST_CLS x = COST_EXTRA y
        const double tok = (double)a / n_ccta;
        double x = (COST_EXTRA * R / extra - tok) / (COST_CLS + COST_EXTRA * n_ccta / extra);
        if (x < 0) x = 0;
        r_cls = (int)(x * n_ccta);
        if (r_cls >= R) { r_cls = R; extra = 0; }
    }
    // entries and rows kept on chip at a time: the expected slice with head-room, and the class CTA's
    // rows, both cut down together when shared memory does not hold them (the kernel then takes its
    // tokens in several stretches)
    long long want_l = (long long)a / n_ccta;
    want_l += want_l / 8 + 64;
    if (want_l > a) want_l = a;
    long long want_r = (r_cls + n_ccta - 1) / n_ccta + 1;
    const long long room = (long long)SMEM_LIMIT - make_layout(sk->n1, 0, 0, G).total - 128;
    const long long need = want_l * (16 + 4 * G) + want_r * 4 * G;     // descriptor + logits per entry, logits per row
    bool cut = false;
    if (need > room) {
        want_l = want_l * room / need;
        want_r = want_r * room / need;
        if (want_l < 2) want_l = 2;
        if (want_r < 1) want_r = 1;
        cut = true;
    }
    want_l = cut ? (want_l & ~1LL) : ((want_l + 1) & ~1LL);       // an even number of entries
    plan->S = S;
    plan->lcap = (int)want_l;
    plan->rcap = (int)want_r;
    plan->extra = extra;
    plan->r_cls = r_cls;
    plan->records = n_ccta + extra;
    const Layout L = make_layout(sk->n1, plan->lcap, plan->rcap, G);
    plan->smem = (size_t)L.total;
    plan->rcap_extra = (L.total - L.wbuf) / (4 * G) - 1;      // a row-only CTA keeps logits where the others keep entries and cells
    return true;
}

cudaError_t kvr_launch_decode_staged(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                                     const void* Kr, const void* Vr, float scale, float* out,
                                     const KvrStagedPlan& plan, float* part, uint32_t* tickets, float* emit,
                                     cudaStream_t st) {
    StagedParams p;
    p.q = q;
    p.Kr = (const uint2*)Kr;
    p.Vr = (const uint2*)Vr;
    p.cells = sk->cells;
    p.clist = sk->clist;
    p.coff = sk->coff;
    p.part = part;
    p.tickets = tickets;
    p.out = out;
    p.status = sk->dev_status;
    p.ml = sk->ml;
    p.inst0 = inst0;
    p.R = rows;
    p.b = sk->d.b;
    p.C = sk->C;
    p.logC = sk->logC;
    p.n1 = sk->n1;
    p.max_ctx = sk->d.max_context;
    p.S = plan.S;
    p.lcap = plan.lcap;
    p.rcap = plan.rcap;
    p.rcap_extra = plan.rcap_extra;
    p.n_ccta = plan.records - plan.extra;
    p.r_cls = plan.r_cls;
    p.zero = 0u;
    p.wait_ns = sk->wait_ns;
    p.tx_extra = sk->tx_extra;
    p.emit = emit;
    p.emit_stride = rows + (N - R);
    p.scale_log2e = scale * 1.4426950408889634f;
    sk->launches += 1;
    const bool f16 = sk->d.kv_dtype == KVR_F16;
    const int gx = plan.records;
    const bool chained = sk->chain && sk->chain_stream == st;
    sk->chain = true;
    sk->chain_stream = st;
#define KVR_STAGED(GG)                                                                                     \
    case GG:                                                                                               \
        if (sk->combine) return f16 ? launch_one<__half, GG, true>(p, n_inst, gx, plan.smem, chained, st)  \
                                    : launch_one<__nv_bfloat16, GG, true>(p, n_inst, gx, plan.smem, chained, st); \
        return f16 ? launch_one<__half, GG, false>(p, n_inst, gx, plan.smem, chained, st)                  \
                   : launch_one<__nv_bfloat16, GG, false>(p, n_inst, gx, plan.smem, chained, st);
    switch (sk->G) {
        KVR_STAGED(1)
        KVR_STAGED(2)
        KVR_STAGED(4)
    }
#undef KVR_STAGED
    return cudaErrorInvalidValue;
}
