// Top-budget selection (Recent + Candidate parts of Algorithm 3, one-shot form) and the copy of
// the retained rows (the exact storage that Algorithm 4 reads back with R.get / C.get).
//
// Selection rule: the newest n_recent tokens are always kept; among the others the R - n_recent
// highest scores are kept, ties broken towards the lower index.  The kernel finds the score of the
// last kept candidate with a 4 x 8-bit radix select over the order-preserving integer image of
// the fp32 scores, then emits both index lists (ascending) and the membership bitmap with ordered
// ballot / warp / CTA prefix counts, so the result is a pure function of the score bits.
#include <cooperative_groups.h>

#include "kvr_internal.h"

namespace cg = cooperative_groups;

namespace {

__device__ __forceinline__ uint32_t score_key(float s) {
    uint32_t u = __float_as_uint(s);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int SEL_THREADS = 1024;
constexpr int SEL_CL = 8;                 // CTAs (one thread-block cluster) per head-instance
constexpr unsigned SEL_FULL = 0xFFFFFFFFu;

// Sum of cnt[w] over the warps w < warp (cnt: one int per warp in shared memory), same value in every lane.
__device__ __forceinline__ int warps_before(const int* cnt, int warp, int lane) {
    int v = (lane < warp) ? cnt[lane] : 0;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(SEL_FULL, v, o);
    return v;
}

// One cluster of SEL_CL CTAs per head-instance; CTA c owns a contiguous range of rows of 32
// consecutive tokens, its warp w a contiguous part of that (lane = token within the row): loads and
// stores are coalesced, a row is one word of the membership bitmap, and ranks within a row come from
// ballots.  The CTAs exchange their digit histograms and their counts through distributed shared
// memory (cluster barriers only; nothing spins).  The scores are re-read (L1/L2) in every pass.
__global__ void __cluster_dims__(SEL_CL, 1, 1) __launch_bounds__(SEL_THREADS, 1)
select_kernel(const float* __restrict__ scores_all, int max_ctx, int inst0, int N, int R, int n_recent,
              int32_t* __restrict__ ret_out, int32_t* __restrict__ cmp_all,
              uint32_t* bitmap_all, int bitmap_words) {
    __shared__ uint32_t hist[2][256];        // this CTA's digit counts (double buffered over the passes)
    __shared__ uint32_t merged[256];         // the cluster's
    __shared__ uint32_t s_prefix, s_krem;
    __shared__ int s_cnt[2][32];
    __shared__ int s_tot[2];                 // this CTA's (threshold ties, kept tokens)

    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int u = blockIdx.y, inst = inst0 + u, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* sc = scores_all + (size_t)inst * max_ctx;
    int32_t* cmp = cmp_all + (size_t)inst * max_ctx;
    uint32_t* bitmap = bitmap_all + (size_t)inst * bitmap_words;
    int32_t* ret = ret_out ? ret_out + (size_t)u * R : nullptr;

    kvr_pdl_trigger();
    kvr_pdl_wait();                      // (as a dependent of the scoring kernel: its scores are complete from here on)
    const int n_cand = N - n_recent;
    const int k = R - n_recent;          // candidates to keep, 0 <= k <= n_cand
    const int rows_cta = ((N + 31) / 32 + SEL_CL - 1) / SEL_CL;
    const int rows = (rows_cta + 31) / 32;                      // rows per warp
    const int r_begin = crank * rows_cta + warp * rows;         // this warp's rows: [r_begin, r_end)
    const int r_end = min(r_begin + rows, (crank + 1) * rows_cta);
    const unsigned lt = (1u << lane) - 1u;
    // f(j, key) for this lane's token of every row of the warp, in order; the scores of four rows are
    // requested before the first of them is used
    auto for_rows = [&](auto&& f) {
        for (int r0 = r_begin; r0 < r_end; r0 += 4) {
            uint32_t key[4];
#pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int j = (r0 + x) * 32 + lane;
                key[x] = (r0 + x < r_end && j < n_cand) ? score_key(sc[j]) : 0u;
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
                if (r0 + x < r_end) f((r0 + x) * 32 + lane, key[x]);              // (uniform condition)
        }
    };

    uint32_t T, k_eq;                    // threshold key; how many keys == T to keep (lowest indices)
    if (k <= 0) {
        T = 0xFFFFFFFFu; k_eq = 0;
    } else if (k >= n_cand) {
        T = 0u; k_eq = 0xFFFFFFFFu;
    } else {
        uint32_t prefix = 0, mask = 0, k_rem = (uint32_t)k;
        for (int pass = 0; pass < 4; ++pass) {
            const int shift = 24 - 8 * pass;
            uint32_t* h = hist[pass & 1];
            if (tid < 256) h[tid] = 0;
            __syncthreads();
            for_rows([&](int j, uint32_t key) {
                const bool act = j < n_cand && (key & mask) == prefix;
                const uint32_t d = (key >> shift) & 255u;
                // Scores of one head share their leading bits, so the lanes of a row fall into very
                // few bins in the first passes: frequent digits are counted with ballots (one
                // addition per digit and row), whatever is left goes to the histogram singly.
                unsigned rem = __ballot_sync(SEL_FULL, act);
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (rem == 0) break;                      // (uniform)
                    const int src = __ffs(rem) - 1;
                    const uint32_t d0 = __shfl_sync(SEL_FULL, d, src);
                    const unsigned m = __ballot_sync(SEL_FULL, act && d == d0);
                    if (lane == src) atomicAdd(&h[d0], (uint32_t)__popc(m));
                    rem &= ~m;
                    if (__popc(m) < 4) break;                 // (uniform) the digits of this row are spread out
                }
                if ((rem >> lane) & 1u) atomicAdd(&h[d], 1u);
            });
            cluster.sync();              // every CTA's counts of this pass are complete
            if (tid < 256) {
                uint32_t tot = 0;
#pragma unroll
                for (int c = 0; c < SEL_CL; ++c) tot += cluster.map_shared_rank(h, c)[tid];
                merged[tid] = tot;
            }
            __syncthreads();
            if (warp == 0) {
                // bins from the top: the first bin at which the running count reaches k_rem
                uint32_t hh[8], tot = 0;
#pragma unroll
                for (int i = 0; i < 8; ++i) { hh[i] = merged[255 - (lane * 8 + i)]; tot += hh[i]; }
                uint32_t inc = tot;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const uint32_t t = __shfl_up_sync(SEL_FULL, inc, o);
                    if (lane >= o) inc += t;
                }
                uint32_t cum = inc - tot;                    // keys in higher bins than this lane's
                const unsigned hit = __ballot_sync(SEL_FULL, inc >= k_rem);
                if (hit != 0 && lane == __ffs(hit) - 1) {    // (the histogram always holds at least k_rem keys)
                    int i = 0;
                    for (; i < 7; ++i) {
                        if (cum + hh[i] >= k_rem) break;
                        cum += hh[i];
                    }
                    s_prefix = prefix | ((uint32_t)(255 - (lane * 8 + i)) << shift);
                    s_krem = k_rem - cum;
                }
            }
            __syncthreads();
            prefix = s_prefix;
            k_rem = s_krem;
            mask |= 0xFFu << shift;
        }
        T = prefix;
        k_eq = k_rem;
    }

    // keys equal to the threshold are kept in index order: count them per warp and per CTA ...
    int n_eq = 0;
    for_rows([&](int j, uint32_t key) { n_eq += __popc(__ballot_sync(SEL_FULL, j < n_cand && key == T)); });
    if (lane == 0) s_cnt[0][warp] = n_eq;
    __syncthreads();
    int eq_before = warps_before(s_cnt[0], warp, lane);
    if (tid == SEL_THREADS - 1) s_tot[0] = eq_before + n_eq;
    cluster.sync();
    for (int c = 0; c < crank; ++c) eq_before += cluster.map_shared_rank(s_tot, c)[0];
    // ... decide every token, one bitmap word per row ...
    int n_keep = 0;
    for_rows([&](int j, uint32_t key) {
        bool keep = false, eq = false;
        if (j < N) {
            if (j >= n_cand) keep = true;
            else {
                keep = key > T;
                eq = key == T;
            }
        }
        const unsigned eqb = __ballot_sync(SEL_FULL, eq);
        if (eq) keep = (uint32_t)(eq_before + __popc(eqb & lt)) < k_eq;
        eq_before += __popc(eqb);
        const unsigned word = __ballot_sync(SEL_FULL, keep);
        if (lane == 0 && j < N) bitmap[j >> 5] = word;
        n_keep += __popc(word);
    });
    if (lane == 0) s_cnt[1][warp] = n_keep;
    __syncthreads();                     // also orders this warp's bitmap words before they are read back
    int keep_before = warps_before(s_cnt[1], warp, lane);
    if (tid == SEL_THREADS - 1) s_tot[1] = keep_before + n_keep;
    cluster.sync();
    for (int c = 0; c < crank; ++c) keep_before += cluster.map_shared_rank(s_tot, c)[1];
    // ... and emit both index lists in ascending order
    for (int r = r_begin; r < r_end; ++r) {
        const int j0 = r * 32, j = j0 + lane;
        if (j0 >= N) break;                                   // (uniform)
        const unsigned word = *reinterpret_cast<volatile uint32_t*>(bitmap + r);
        const int pos = keep_before + __popc(word & lt);      // kept tokens before j
        if (j < N) {
            if ((word >> lane) & 1u) { if (ret) ret[pos] = j; }
            else cmp[j - pos] = j;
        }
        keep_before += __popc(word);
    }
    cluster.sync();                      // no CTA leaves while another may still read its shared memory
}

// 16 threads per row, 16 bytes each: rows of 128 16-bit elements.
__global__ void gather_kernel(const uint4* __restrict__ K, const uint4* __restrict__ V,
                              const int32_t* __restrict__ ret_idx, int N, int R, uint4* __restrict__ Kr,
                              uint4* __restrict__ Vr) {
    const int u = blockIdx.y;
    const int row = blockIdx.x * (blockDim.x >> 4) + (threadIdx.x >> 4);
    const int c = threadIdx.x & 15;
    kvr_pdl_trigger();
    kvr_pdl_wait();                      // (as a dependent of the selection: the index list is complete from here on)
    if (row >= R) return;
    const int J = ret_idx[(size_t)u * R + row];
    const size_t src = ((size_t)u * N + J) * 16 + c, dst = ((size_t)u * R + row) * 16 + c;
    Kr[dst] = K[src];
    Vr[dst] = V[src];
}

}  // namespace

cudaError_t kvr_launch_select(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int n_recent,
                              int32_t* ret_idx, cudaStream_t st) {
    // (follows the scoring kernels of the same compress on `st`)
    const cudaError_t e = kvr_launch_after(select_kernel, dim3(SEL_CL, n_inst), dim3(SEL_THREADS), 0, st, true, (const float*)sk->scores,
                                           sk->d.max_context, inst0, N, R, n_recent, ret_idx, sk->cmp_idx, sk->bitmap,
                                           sk->bitmap_words);
    sk->launches += 1;
    return e;
}

// The same selection on caller-provided scores of `n` stored rows (stride n): positions kept
// (ascending) -> keep_pos [n_inst][R], the others -> rest_pos [n_inst][n], membership of positions -> bits.
cudaError_t kvr_launch_select_rows(kvr_sketch* sk, const float* scores, int n, int n_inst, int R, int n_recent,
                                   int32_t* keep_pos, int32_t* rest_pos, uint32_t* bits, int words, cudaStream_t st) {
    select_kernel<<<dim3(SEL_CL, n_inst), SEL_THREADS, 0, st>>>(scores, n, 0, n, R, n_recent, keep_pos, rest_pos, bits, words);
    sk->launches += 1;
    return cudaGetLastError();
}

cudaError_t kvr_launch_gather(kvr_sketch* sk, int n_inst, int N, int R, const void* K, const void* V,
                              const int32_t* ret_idx, void* Kr, void* Vr, cudaStream_t st) {
    if (R <= 0) return cudaSuccess;
    dim3 g((R + 15) / 16, n_inst);
    const cudaError_t e = kvr_launch_after(gather_kernel, g, dim3(256), 0, st, true, (const uint4*)K, (const uint4*)V, ret_idx, N, R,
                                           (uint4*)Kr, (uint4*)Vr);
    sk->launches += 1;
    return e;
}
