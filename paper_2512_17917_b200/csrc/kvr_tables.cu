// Integer side of the sketch: hash / sign tables over token indices (built once per handle),
// cell -> token lists, and the per-head-instance list of compressed tokens that the decode
// kernels walk.  Everything here is exact integer work.
//
// Hash family (Vague Sketch section, Algorithms 1-2 leave h_i, g_i open):
//   h_i(J) = ((A_i m(J) + C_i) mod p) mod b,  g_i(J) = +1/-1 for (A'_i m(J) + C'_i) mod p even/odd,
//   p = 2^31 - 1, m = fixed 32-bit scrambling bijection (or the identity in test mode).
#include <cooperative_groups.h>

#include "kvr_internal.h"

namespace cg = cooperative_groups;

namespace {

struct SeedPack {
    uint32_t s[KVR_R_MAX][4];
};

__device__ __forceinline__ uint32_t mix_index(uint32_t x, int mix) {
    if (!mix) return x;
    x ^= x >> 16;
    x *= 0x85EBCA6Bu;
    x ^= x >> 13;
    x *= 0xC2B2AE35u;
    x ^= x >> 16;
    return x;
}

// x mod (2^31 - 1) for x < 2^63, by folding 31-bit digits (2^31 = 1 mod p).
__device__ __forceinline__ uint32_t mod_p(uint64_t x) {
    uint64_t y = (x & KVR_HASH_P) + (x >> 31);        // < 2^32 + 2^31
    y = (y & KVR_HASH_P) + (y >> 31);                 // <= p + 2
    if (y >= KVR_HASH_P) y -= KVR_HASH_P;
    return (uint32_t)y;
}

__global__ void hash_table_kernel(SeedPack sp, int r, int mix, int b, int max_ctx, int32_t* __restrict__ tok_h,
                                  int8_t* __restrict__ tok_g, uint32_t* __restrict__ tok_pack) {
    int J = blockIdx.x * blockDim.x + threadIdx.x;
    if (J >= max_ctx) return;
    uint64_t m = mix_index((uint32_t)J, mix);
    uint32_t h[KVR_R_MAX], neg[KVR_R_MAX];
#pragma unroll
    for (int i = 0; i < KVR_R_MAX; ++i) {
        if (i >= r) { h[i] = 0; neg[i] = 0; continue; }
        uint32_t x = mod_p((uint64_t)sp.s[i][0] * m + sp.s[i][1]);
        h[i] = x % (uint32_t)b;
        uint32_t y = mod_p((uint64_t)sp.s[i][2] * m + sp.s[i][3]);
        neg[i] = y & 1u;
        tok_h[(size_t)i * max_ctx + J] = (int32_t)h[i];
        tok_g[(size_t)i * max_ctx + J] = neg[i] ? (int8_t)-1 : (int8_t)1;
    }
    if (r == KVR_R) tok_pack[J] = h[1] | (h[2] << KVR_PACK_H2_SHIFT) |
                  ((neg[0] | (neg[1] << 1) | (neg[2] << 2)) << KVR_PACK_SIGN_SHIFT);
}

// One thread per (row, cell): count the tokens of the cell.
__global__ void csr_count_kernel(const int32_t* __restrict__ tok_h, int b, int max_ctx,
                                 int32_t* __restrict__ cnt /*[r][b]*/) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    int i = blockIdx.y;
    if (c >= b) return;
    const int32_t* h = tok_h + (size_t)i * max_ctx;
    int n = 0;
    for (int J = 0; J < max_ctx; ++J) n += (h[J] == c);
    cnt[i * b + c] = n;
}

// One CTA per row: exclusive scan of the b counts (b <= 8192).
__global__ void csr_scan_kernel(const int32_t* __restrict__ cnt, int b, int32_t* __restrict__ off /*[r][b+1]*/) {
    __shared__ int32_t part[1024];
    int i = blockIdx.x, tid = threadIdx.x, nt = blockDim.x;
    int per = (b + nt - 1) / nt;
    int lo = tid * per, hi = min(lo + per, b);
    int s = 0;
    for (int c = lo; c < hi; ++c) s += cnt[i * b + c];
    part[tid] = s;
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int t = 0; t < nt; ++t) {
            int v = part[t];
            part[t] = run;
            run += v;
        }
    }
    __syncthreads();
    int run = part[tid];
    for (int c = lo; c < hi; ++c) {
        off[i * (b + 1) + c] = run;
        run += cnt[i * b + c];
    }
    if (hi == b && lo <= b) off[i * (b + 1) + b] = run;   // the thread that ends at b writes the total
}

// One thread per (row, cell): write the cell's tokens in ascending order.
__global__ void csr_fill_kernel(const int32_t* __restrict__ tok_h, const int32_t* __restrict__ off, int b,
                                int max_ctx, int32_t* __restrict__ list /*[r][max_ctx]*/) {
    int c = blockIdx.x * blockDim.x + threadIdx.x;
    int i = blockIdx.y;
    if (c >= b) return;
    const int32_t* h = tok_h + (size_t)i * max_ctx;
    int32_t* out = list + (size_t)i * max_ctx;
    int p = off[i * (b + 1) + c];
    for (int J = 0; J < max_ctx; ++J)
        if (h[J] == c) out[p++] = J;
}

// Per head-instance, the token lists the decode kernels walk:
//   dlist / doff   the compressed tokens (index < N and not retained by the membership bitmap) in
//                  row-0-cell order, ascending token index inside a cell, as packed entries
//   clist / coff / ctok  (when the handle has a class grid, C > 0) the same tokens regrouped into C x C
//                  classes by (row-1 cell mod C, row-2 cell mod C), row-0-cell order kept inside each
//                  class, the first token of every row-0 cell inside its class flagged and told the
//                  row-0 cell of the run that follows it
// One cluster of LST_CL CTAs per head-instance; CTA r owns a contiguous range of row-0 cells, one
// warp a cell at a time.  Pass 1 counts the kept tokens per (cell, class); the CTAs exchange their
// column sums through distributed shared memory (cluster barriers, nothing spins); ordered scans turn
// the counts into positions; pass 2 walks the cells again and writes both lists.  Every position is
// a pure function of the inputs (ballot / match ranks and ordered sums), not of the scheduling.
constexpr int LST_CL = 8, LST_THREADS = 1024;

__global__ void __cluster_dims__(LST_CL, 1, 1) __launch_bounds__(LST_THREADS, 1)
lists_kernel(const int32_t* __restrict__ full_off, const int32_t* __restrict__ full_list,
             const uint32_t* __restrict__ tok_pack, const uint32_t* __restrict__ bitmap_all, int bitmap_words,
             int b, int N, int max_ctx, int inst0, int n_tbl, int C, int logC, int n1, uint32_t* __restrict__ dlist_all,
             int32_t* __restrict__ doff_all, uint2* __restrict__ clist_all, int32_t* __restrict__ coff_all,
             int32_t* __restrict__ ctok_all) {
    extern __shared__ int32_t s_cnt[];        // [cells of this CTA][1 + C * C]: kept tokens, then per class
    __shared__ int32_t s_tot[65];             // column sums over this CTA's cells
    __shared__ int32_t s_all[65];             // column sums over the cluster
    __shared__ int32_t s_base[65];            // position of this CTA's first entry of each column
    __shared__ int32_t s_run[32][64];         // per warp: entries of the current cell already written, per class

    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank();
    const int inst = inst0 + blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    {
        const int tb = n_tbl > 1 ? inst % n_tbl : 0;            // hash tables of this kv head, or the shared ones
        full_off += (size_t)tb * KVR_R * (b + 1);
        full_list += (size_t)tb * KVR_R * max_ctx;
        tok_pack += (size_t)tb * max_ctx;
    }
    const int n_cls = C * C, n_col = 1 + n_cls;
    const int bc = (b + LST_CL - 1) / LST_CL;
    const int c_lo = min(crank * bc, b), c_hi = min(c_lo + bc, b), n_c = c_hi - c_lo;
    const unsigned lt = (1u << lane) - 1u;
    const uint32_t* bitmap = bitmap_all + (size_t)inst * bitmap_words;
    uint32_t* dlist = dlist_all + (size_t)inst * max_ctx;
    int32_t* doff = doff_all + (size_t)inst * (b + 1);

    auto cls = [&](uint32_t e) {
        const uint32_t h1 = e & KVR_PACK_H_MASK, h2 = (e >> KVR_PACK_H2_SHIFT) & KVR_PACK_H_MASK;
        return (int)(((h1 & (C - 1)) << logC) | (h2 & (C - 1)));
    };
    // this lane's tokens of the 4 x 32 list positions starting at `base` of a cell that ends at p1: the four
    // token indices are asked for together, then their membership words and packed cells together (two
    // round trips to memory per 128 positions instead of three per 32)
    constexpr int LST_PF = 4;
    auto fetch = [&](int base, int p1, bool (&keep)[LST_PF], uint32_t (&e)[LST_PF], int (&J)[LST_PF]) {
#pragma unroll
        for (int x = 0; x < LST_PF; ++x) {
            const int p = base + 32 * x + lane;
            J[x] = (p < p1) ? full_list[p] : N;
        }
        uint32_t w[LST_PF];
#pragma unroll
        for (int x = 0; x < LST_PF; ++x) {
            const bool in = J[x] < N;
            w[x] = in ? bitmap[J[x] >> 5] : 0xFFFFFFFFu;
            e[x] = in ? tok_pack[J[x]] : 0u;
        }
#pragma unroll
        for (int x = 0; x < LST_PF; ++x) {
            keep[x] = (J[x] < N) && !((w[x] >> (J[x] & 31)) & 1u);
            if (!keep[x]) { e[x] = 0u; J[x] = 0; }
        }
    };

    // ---- pass 1: counts per (cell, column)
    for (int idx = tid; idx < n_c * n_col; idx += LST_THREADS) s_cnt[idx] = 0;
    __syncthreads();
    for (int c = c_lo + warp; c < c_hi; c += 32) {
        const int p0 = full_off[c], p1 = full_off[c + 1];
        int32_t* row = s_cnt + (size_t)(c - c_lo) * n_col;
        int n = 0;
        for (int base4 = p0; base4 < p1; base4 += 32 * LST_PF) {          // warp-uniform trip counts
            bool keep4[LST_PF];
            uint32_t e4[LST_PF];
            int J4[LST_PF];
            fetch(base4, p1, keep4, e4, J4);
#pragma unroll
            for (int x = 0; x < LST_PF; ++x) {
                if (base4 + 32 * x >= p1) break;
                const bool keep = keep4[x];
                const uint32_t e = e4[x];
                n += __popc(__ballot_sync(0xFFFFFFFFu, keep));
                if (n_cls) {
                    const int k = keep ? cls(e) : 64;
                    const unsigned same = __match_any_sync(0xFFFFFFFFu, k);
                    if (keep && (same & lt) == 0u) row[1 + k] += __popc(same);   // lowest lane of each class present
                    __syncwarp();
                }
            }
        }
        if (lane == 0) row[0] = n;
    }
    __syncthreads();
    // ---- column sums of this CTA, exchanged over the cluster
    for (int col = warp; col < n_col; col += 32) {
        int v = 0;
        for (int c = lane; c < n_c; c += 32) v += s_cnt[(size_t)c * n_col + col];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
        if (lane == 0) s_tot[col] = v;
    }
    cluster.sync();
    if (tid < n_col) {
        int all = 0, before = 0;
        for (int r = 0; r < LST_CL; ++r) {
            const int v = cluster.map_shared_rank(s_tot, r)[tid];
            all += v;
            if (r < crank) before += v;
        }
        s_all[tid] = all;
        s_base[tid] = before;
    }
    __syncthreads();
    if (tid >= 1 && tid < n_col) {                            // class k = tid - 1 starts after all lower classes
        int lower = 0;
        for (int k = 1; k < tid; ++k) lower += s_all[k];
        if (crank == 0) coff_all[(size_t)inst * (n_cls + 1) + (tid - 1)] = lower;
        s_base[tid] += lower;                                 // (only this thread touches s_base[tid])
    }
    if (tid == 0) {
        if (crank == 0 && n_cls) coff_all[(size_t)inst * (n_cls + 1) + n_cls] = s_all[0];
        if (crank == LST_CL - 1) doff[b] = s_all[0];
    }
    __syncthreads();
    // ---- counts -> positions: ordered scan over this CTA's cells, one warp per column
    for (int col = warp; col < n_col; col += 32) {
        int run = s_base[col];
        for (int c0 = 0; c0 < n_c; c0 += 32) {
            const int c = c0 + lane;
            const int v = (c < n_c) ? s_cnt[(size_t)c * n_col + col] : 0;
            int inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int t = __shfl_up_sync(0xFFFFFFFFu, inc, o);
                if (lane >= o) inc += t;
            }
            if (c < n_c) {
                s_cnt[(size_t)c * n_col + col] = run + inc - v;
                if (col == 0) doff[c_lo + c] = run + inc - v;
            }
            run += __shfl_sync(0xFFFFFFFFu, inc, 31);
        }
    }
    __syncthreads();
    // ---- pass 2: write the lists
    uint2* cl = n_cls ? clist_all + (size_t)inst * max_ctx : nullptr;
    int32_t* ct = n_cls ? ctok_all + (size_t)inst * max_ctx : nullptr;
    for (int c = c_lo + warp; c < c_hi; c += 32) {
        const int p0 = full_off[c], p1 = full_off[c + 1];
        const int32_t* row = s_cnt + (size_t)(c - c_lo) * n_col;
        if (n_cls) {
            for (int k = lane; k < n_cls; k += 32) s_run[warp][k] = 0;
            __syncwarp();
        }
        int w = row[0];
        for (int base4 = p0; base4 < p1; base4 += 32 * LST_PF) {
          bool keep4[LST_PF];
          uint32_t e4[LST_PF];
          int J4[LST_PF];
          fetch(base4, p1, keep4, e4, J4);
#pragma unroll
          for (int x = 0; x < LST_PF; ++x) {
            if (base4 + 32 * x >= p1) break;
            const bool keep = keep4[x];
            const uint32_t e = e4[x];
            const int J = J4[x];
            const unsigned m = __ballot_sync(0xFFFFFFFFu, keep);
            if (keep) dlist[w + __popc(m & lt)] = e;
            w += __popc(m);
            if (n_cls) {
                const int k = keep ? cls(e) : 64;
                const unsigned same = __match_any_sync(0xFFFFFFFFu, k);
                if (keep) {
                    const int seen = s_run[warp][k] + __popc(same & lt);    // tokens of (cell, class) before this one
                    const uint32_t h1 = e & KVR_PACK_H_MASK, h2 = (e >> KVR_PACK_H2_SHIFT) & KVR_PACK_H_MASK;
                    const uint32_t sg = e >> KVR_PACK_SIGN_SHIFT;
                    const uint32_t s3 = (sg & 1u) | (((sg ^ (sg >> 1)) & 1u) << 1) | (((sg ^ (sg >> 2)) & 1u) << 2);
                    cl[row[1 + k] + seen] = make_uint2((h1 >> logC) | (((uint32_t)n1 + (h2 >> logC)) << 8),
                                                       ((uint32_t)c << KVR_CL_C0_SHIFT) | (s3 << KVR_CL_SIGN_SHIFT) |
                                                           (seen == 0 ? KVR_CL_FLAG : 0u));
                    ct[row[1 + k] + seen] = J;
                }
                __syncwarp();
                if (keep && (same & lt) == 0u) s_run[warp][k] += __popc(same);
                __syncwarp();
            }
          }
        }
    }
    cluster.sync();                      // no CTA leaves while another may still read its column sums;
                                         // every entry of the class list is written and visible
    // ---- pass 3: every entry learns the row-0 cell of the next flagged entry of the list (flagged =
    // first token of a row-0 cell inside its class), which is the cell the decode kernel fetches ahead
    // while it works on the entry's run.  The first entry of every class is flagged, so a walk ends at
    // the next class's first entry at the latest; the last run of the list names its own cell.
    if (n_cls) {
        const int a = s_all[0];
        for (int i = crank * LST_THREADS + tid; i < a; i += LST_CL * LST_THREADS) {
            const uint2 e = cl[i];
            if (!(e.y & KVR_CL_FLAG)) continue;
            int j = i + 1;
            while (j < a && !(cl[j].y & KVR_CL_FLAG)) ++j;
            const uint32_t nxt = ((j < a ? cl[j].y : e.y) >> KVR_CL_C0_SHIFT) << KVR_CL_NEXT_SHIFT;
            for (int k = i; k < j; ++k) cl[k].x = (cl[k].x & 0xFFFFu) | nxt;
        }
    }
}

__global__ void assignment_kernel(const int32_t* __restrict__ cmp_all, const int32_t* __restrict__ tok_h,
                                  const int8_t* __restrict__ tok_g, int r, int max_ctx, int a, int inst0, int n_tbl,
                                  int32_t* __restrict__ cmp_out, int32_t* __restrict__ bucket,
                                  int8_t* __restrict__ sign) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    int u = blockIdx.y;
    if (t >= a) return;
    const int tb = n_tbl > 1 ? (inst0 + u) % n_tbl : 0;
    tok_h += (size_t)tb * r * max_ctx;
    tok_g += (size_t)tb * r * max_ctx;
    int J = cmp_all[(size_t)(inst0 + u) * max_ctx + t];
    if (cmp_out) cmp_out[(size_t)u * a + t] = J;
    for (int i = 0; i < r; ++i) {
        if (bucket) bucket[((size_t)u * r + i) * a + t] = tok_h[(size_t)i * max_ctx + J];
        if (sign) sign[((size_t)u * r + i) * a + t] = tok_g[(size_t)i * max_ctx + J];
    }
}

}  // namespace

cudaError_t kvr_launch_hash_tables(kvr_sketch* sk, cudaStream_t st) {
    const int b = sk->d.b, mc = sk->d.max_context, r = sk->d.r;
    int32_t* cnt = nullptr;
    cudaError_t e = cudaMalloc(&cnt, sizeof(int32_t) * r * b);
    if (e != cudaSuccess) return e;
    for (int t = 0; t < sk->n_tbl; ++t) {                       // one set of tables per kv head, or one for all
        SeedPack sp = {};
        for (int i = 0; i < r; ++i)
            for (int k = 0; k < 4; ++k) sp.s[i][k] = sk->seeds[((size_t)t * r + i) * 4 + k];
        int32_t* tok_h = sk->tok_h + (size_t)t * r * mc;
        int8_t* tok_g = sk->tok_g + (size_t)t * r * mc;
        int32_t* full_off = sk->full_off + (size_t)t * r * (b + 1);
        int32_t* full_list = sk->full_list + (size_t)t * r * mc;
        hash_table_kernel<<<(mc + 255) / 256, 256, 0, st>>>(sp, r, sk->d.index_mix, b, mc, tok_h, tok_g,
                                                            sk->tok_pack + (size_t)t * mc);
        dim3 g((b + 127) / 128, r);
        csr_count_kernel<<<g, 128, 0, st>>>(tok_h, b, mc, cnt);
        csr_scan_kernel<<<r, 1024, 0, st>>>(cnt, b, full_off);
        csr_fill_kernel<<<g, 128, 0, st>>>(tok_h, full_off, b, mc, full_list);
        sk->launches += 4;
    }
    e = cudaStreamSynchronize(st);
    cudaFree(cnt);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// dlist / doff always; clist / coff when the handle has a class grid.
cudaError_t kvr_launch_lists(kvr_sketch* sk, int inst0, int n_inst, int N, cudaStream_t st) {
    const int b = sk->d.b, C = sk->C > 0 ? sk->C : 0;
    const int bc = (b + LST_CL - 1) / LST_CL;
    const size_t smem = sizeof(int32_t) * (size_t)bc * (1 + C * C);
    lists_kernel<<<dim3(LST_CL, n_inst), LST_THREADS, smem, st>>>(sk->full_off, sk->full_list, sk->tok_pack, sk->bitmap,
                                                                  sk->bitmap_words, b, N, sk->d.max_context, inst0, sk->n_tbl, C,
                                                                  sk->logC, sk->n1, sk->dlist, sk->doff, sk->clist,
                                                                  sk->coff, sk->ctok);
    sk->launches += 1;
    return cudaGetLastError();
}

cudaError_t kvr_launch_assignment(const kvr_sketch* sk, int inst0, int n_inst, int a, int32_t* cmp_idx,
                                  int32_t* bucket, int8_t* sign, cudaStream_t st) {
    if (a <= 0 || n_inst <= 0) return cudaSuccess;
    dim3 g((a + 255) / 256, n_inst);
    assignment_kernel<<<g, 256, 0, st>>>(sk->cmp_idx, sk->tok_h, sk->tok_g, sk->d.r, sk->d.max_context, a, inst0, sk->n_tbl,
                                         cmp_idx, bucket, sign);
    const_cast<kvr_sketch*>(sk)->launches += 1;
    return cudaGetLastError();
}
