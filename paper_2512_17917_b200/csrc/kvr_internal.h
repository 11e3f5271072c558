// Internal declarations shared by the host layer (kvr_api.cu) and the kernel files of libkvr.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

#include "kvr.h"

#define KVR_D 128       // head_dim the kernels are written for
#define KVR_R 3         // sketch rows the fast kernels are written for (the paper's fixed value)
#define KVR_R_MAX 5     // rows the general kernels accept (1, 3 or 5)
#define KVR_HASH_P 2147483647ull

// Per compressed token, packed for the decode kernels: bits 0-12 = cell of row 1, bits 13-25 =
// cell of row 2, bits 26-28 = 1 where g_0 / g_1 / g_2 is -1.  (The row-0 cell is implied by the
// position of the entry in the row-0-ordered list.)
#define KVR_PACK_H2_SHIFT 13
#define KVR_PACK_SIGN_SHIFT 26
#define KVR_PACK_H_MASK 0x1FFFu

// Per compressed token, for the staged decode kernel (tokens grouped by class, see kvr_sketch::C):
//   x: bits 0-7 = index of the row-1 cell inside the class's slice, bits 8-15 = index of the row-2
//      cell inside the staged array (row-2 slice follows the row-1 slice; the array has at most 226
//      cells of 1 KB), bits 16-31 = row-0 cell of the next flagged entry of the list (the cell
//      the kernel fetches ahead while it works on this entry's run)
//   y: bit 0 = first token of its row-0 cell inside its class (the row-0 cell must be reloaded),
//      bit 4 = g_0 is -1, bit 5 = g_0 g_1 is -1, bit 6 = g_0 g_2 is -1 (so that y & 0x70 is the byte
//      offset of a 16-byte row in a table of sign pairs), bits 16-31 = row-0 cell
#define KVR_CL_FLAG 1u
#define KVR_CL_SIGN_SHIFT 4
#define KVR_CL_C0_SHIFT 16
#define KVR_CL_NEXT_SHIFT 16

struct kvr_sketch {
    kvr_sketch_desc_t d;
    int G;           // query heads per kv head
    int BH;          // batch * n_kv_heads = head-instances per layer
    int n_inst;      // BH * n_layers
    int device;
    int n_sm;
    int n_tbl;       // sets of hash tables: 1 (seeds shared by all heads) or n_kv_heads (seeds per kv head)
    std::vector<uint32_t> seeds;   // [n_tbl][r][4]

    // ---- per-handle hash tables over token indices 0 .. max_context-1 (device) ----
    int32_t* tok_h;      // [n_tbl][r][max_context]   cell of token J in row i
    int8_t* tok_g;       // [r][max_context]   +1 / -1
    uint32_t* tok_pack;  // [max_context]      packed rows 1,2 + signs (see above)
    int32_t* full_off;   // [r][b+1]           CSR offsets: tokens of each cell, ascending
    int32_t* full_list;  // [r][max_context]

    // ---- per head-instance state (device) ----
    float* cells;        // [n_inst][2][r][b][D]
    float* scores;       // [n_inst][max_context]
    int32_t* cmp_idx;    // [n_inst][max_context]  compressed tokens ascending
    uint32_t* bitmap;    // [n_inst][bitmap_words] bit J set = token J retained
    uint32_t* dlist;     // [n_inst][max_context]  packed entries of compressed tokens, row-0 cell order
    int32_t* doff;       // [n_inst][b+1]          offsets of each row-0 cell in dlist
    // Staged decode kernel: tokens are split into C x C classes by (row-1 cell mod C, row-2 cell mod C)
    // so that the cells one class touches in rows 1 and 2 fit in one SM's shared memory.
    int C, logC, n1;     // C = 0: sketch too wide for the staged kernel; n1 = ceil(b / C)
    uint2* clist;        // [n_inst][max_context]  class-ordered entries (format above)
    int32_t* coff;       // [n_inst][C*C+1]        offsets of each class in clist
    int32_t* ctok;       // [n_inst][max_context]  token index of each clist entry
    int bitmap_words;

    // ---- per layer host state ----
    std::vector<int32_t> layer_N, layer_R;  // -1 = never compressed

    // ---- workspaces (device, grown on demand) ----
    void* ws_score;  size_t ws_score_bytes;   // score partial row statistics
    void* ws_decode; size_t ws_decode_bytes;  // split partials
    uint32_t* tickets;                        // [n_inst] arrival counters, zero between calls
    int32_t* dev_status;                      // device word: non-zero after a kernel's bounded wait gave up
    float* ml;                                // [n_inst][G][2] softmax reference maximum (log2 units) and sum of
                                              // the last decode of each head-instance (for score accumulation)
    void* ws_demote; size_t ws_demote_bytes;  // positions / membership of the overflow step
    void* ws_emit; size_t ws_emit_bytes;      // logits the staged kernel emits for the scored decode call
    void* ws_append; size_t ws_append_bytes;  // storage + new rows before the overflow step of kvr_append

    // ---- host-buffer path (allocated on first use) ----
    void* st_K; void* st_V; void* st_Q; size_t st_k_bytes, st_v_bytes, st_q_bytes;
    void* st_Kr; void* st_Vr; int32_t* st_ret; size_t st_ret_rows;   // retained store [n_inst][st_ret_rows][D]
    void* st_q1; void* st_out; size_t st_q1_bytes, st_out_bytes;

    // ---- decode kernel choice ----
    int decode_kernel;       // kvr_decode_kernel_t requested by the caller
    int last_decode_kernel;  // which kernel the last decode call launched (KVR_DECODE_SPLIT / _STAGED)
    unsigned long long wait_ns;   // limit of the staged decode kernel's waits on its staging barriers
    uint32_t tx_extra;       // bytes the staged kernel announces beyond what it copies (test hook; 0)
    int score_kernel;        // kvr_score_kernel_t requested by the caller
    int obs_causal;          // observation window inside the context, causally masked
    int combine;             // kvr_combine_t: 0 = element-wise median of the three cells, 1 = their mean
    bool chain;              // the last kernel that touched the handle was a staged decode launch on chain_stream
    cudaStream_t chain_stream;   // and no call has changed cells or token lists since
    int last_score_kernel;   // which scoring kernels the last compress launched

    // ---- side stream: the token lists are built while the sketch insertion runs ----
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;

    size_t device_bytes;
    int64_t launches;
};

// How the staged decode kernel runs one call.
struct KvrStagedPlan {
    int S;         // token slices per class
    int lcap;      // token entries staged at a time
    int rcap;      // retained rows of a class CTA whose logits are kept on chip at a time
    int rcap_extra;  // the same for a CTA that only streams rows
    int extra;     // CTAs per head-instance that only stream retained rows (SMs the classes leave idle)
    int r_cls;     // retained rows handled by the class CTAs (the rest go to the extra CTAs)
    int records;   // partial records per head-instance (C*C*S + extra)
    size_t smem;   // dynamic shared memory per CTA
};

// ---- kernel launchers (each returns the cudaError_t of its launches) --------------------------
struct ScoreShape {
    int n_inst;     // instances in this call
    int inst0;      // first instance (index into handle arrays)
    int N, M;       // keys, observation rows per instance (G*W)
    int W;          // observation queries per head
    int causal;     // the W queries are the last W context tokens: query t sees the keys <= N - W + t
    int chunk;      // keys per CTA (multiple of 64)
    int n_chunks;
    float scale_log2e;
};

cudaError_t kvr_launch_hash_tables(kvr_sketch* sk, cudaStream_t st);
cudaError_t kvr_launch_scores(kvr_sketch* sk, const ScoreShape& s, const void* K, const void* Q,
                              cudaStream_t st);
// tcgen05 scoring: availability for a shape, its chunking (fills chunk / n_chunks), its workspace
bool kvr_scores_tc_supported(const ScoreShape& s, const void* K, const void* Q);
void kvr_scores_tc_plan(const kvr_sketch* sk, ScoreShape* s);
size_t kvr_scores_tc_ws_bytes(const ScoreShape& s);
cudaError_t kvr_launch_scores_tc(kvr_sketch* sk, const ScoreShape& s, const void* K, const void* Q,
                                 cudaStream_t st);
cudaError_t kvr_launch_select(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int n_recent,
                              int32_t* ret_idx, cudaStream_t st);
cudaError_t kvr_launch_select_rows(kvr_sketch* sk, const float* scores, int n, int n_inst, int R, int n_recent,
                                   int32_t* keep_pos, int32_t* rest_pos, uint32_t* bits, int words, cudaStream_t st);
cudaError_t kvr_launch_gather(kvr_sketch* sk, int n_inst, int N, int R, const void* K, const void* V,
                              const int32_t* ret_idx, void* Kr, void* Vr, cudaStream_t st);
cudaError_t kvr_launch_insert(kvr_sketch* sk, int inst0, int n_inst, int N, const void* K,
                              const void* V, cudaStream_t st);
cudaError_t kvr_launch_lists(kvr_sketch* sk, int inst0, int n_inst, int N, cudaStream_t st);
// N, R: context length and retained count of the layer's compress; rows >= R: rows of Kr / Vr per
// head-instance (the R retained tokens followed by tokens appended after the compress)
cudaError_t kvr_launch_decode(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                              const void* Kr, const void* Vr, float scale, float* out, int n_splits,
                              cudaStream_t st);
cudaError_t kvr_launch_reconstruct(const kvr_sketch* sk, int inst0, int n_inst, int a, float* Kt,
                                   float* Vt, cudaStream_t st);
cudaError_t kvr_launch_assignment(const kvr_sketch* sk, int inst0, int n_inst, int a, int32_t* cmp_idx,
                                  int32_t* bucket, int8_t* sign, cudaStream_t st);

cudaError_t kvr_launch_decode_generic(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                                      const void* Kr, const void* Vr, float scale, float* out, int n_splits,
                                      cudaStream_t st);
cudaError_t kvr_launch_reconstruct_generic(const kvr_sketch* sk, int inst0, int n_inst, int a, float* Kt, float* Vt,
                                           cudaStream_t st);

int kvr_decode_staged_pick_C(int b, int G);
bool kvr_decode_staged_plan(const kvr_sketch* sk, int n_inst, int N, int R, int rows, bool forced, KvrStagedPlan* plan);
cudaError_t kvr_launch_decode_staged(kvr_sketch* sk, int inst0, int n_inst, int N, int R, int rows, const void* q,
                                     const void* Kr, const void* Vr, float scale, float* out,
                                     const KvrStagedPlan& plan, float* part, uint32_t* tickets, float* emit,
                                     cudaStream_t st);
// emit (or null): [n_inst][rows + (N - R)][G] logits (log2 units) of the rows, then of the class-list entries;
// kvr_launch_apply_emitted turns them into attention mass under the launch's final (max, sum) and adds the
// rows' to score_acc [n_inst][rows], the tokens' to the handle's per-token scores.
cudaError_t kvr_launch_apply_emitted(kvr_sketch* sk, int inst0, int n_inst, int rows, int a, const float* emit,
                                     float* score_acc, cudaStream_t st);
// attention mass of the rows of Kr under the softmax of the layer's last decode, added to acc
cudaError_t kvr_launch_row_mass(kvr_sketch* sk, int inst0, int n_inst, int rows, const void* q, const void* Kr,
                                float scale, float* acc, cudaStream_t st);
// overflow step: rows -> kept rows + sketch (see kvr_demote in kvr.h); ws = workspace of kvr_demote_ws_bytes
size_t kvr_demote_ws_bytes(int n_inst, int rows);
cudaError_t kvr_launch_vague_mass(kvr_sketch* sk, int inst0, int n_inst, int a, const void* q, float scale,
                                  cudaStream_t st);
cudaError_t kvr_launch_swap(kvr_sketch* sk, int inst0, int n_inst, int N, int a, void* Kr, void* Vr, int32_t* ret_idx,
                            float* row_scores, int rows, int n_recent, float rate, int max_swaps, int32_t* n_swapped,
                            cudaStream_t st);
cudaError_t kvr_launch_demote(kvr_sketch* sk, int inst0, int n_inst, int rows, int N_new, int budget, int n_recent,
                              const void* Kr, const void* Vr, const int32_t* ret_idx, const float* row_scores,
                              void* Kr_out, void* Vr_out, int32_t* ret_out, float* scores_out, void* ws,
                              cudaStream_t st);

cudaError_t kvr_launch_append_rows(kvr_sketch* sk, int n_inst, const void* Kr, const void* Vr, const int32_t* ret,
                                   const float* rs, int rows, const void* Kn, const void* Vn, int n_new, int ctx0,
                                   void* Ko, void* Vo, int32_t* ro, float* so, cudaStream_t st);

// several queries per head (kvr_decode_mq.cu)
bool kvr_decode_mq_plan(const kvr_sketch* sk, int n_inst, int N, int R, int* S_out, int* lcap_out, size_t* smem_out);
size_t kvr_decode_mq_ws_bytes(int n_inst, int records);
cudaError_t kvr_launch_decode_mq(kvr_sketch* sk, int inst0, int n_inst, int rows, const void* q, const void* Kr, const void* Vr,
                                 int n_queries, int causal, float scale, float* out, int S, int lcap, size_t smem, float* part,
                                 cudaStream_t st);

size_t kvr_decode_ws_bytes(int n_inst, int n_splits, int G);
int kvr_decode_pick_splits(const kvr_sketch* sk, int n_inst, int N, int R);

// ---- small device helpers ---------------------------------------------------------------------
#ifdef __CUDACC__
template <typename T> struct KvrType;
template <> struct KvrType<__half> {
    using v2 = __half2;
    static __device__ __forceinline__ float2 to_f2(uint32_t u) {
        return __half22float2(*reinterpret_cast<const __half2*>(&u));
    }
    static __device__ __forceinline__ float to_float(__half x) { return __half2float(x); }
    static __device__ __forceinline__ __half from_float(float x) { return __float2half_rn(x); }
};
template <> struct KvrType<__nv_bfloat16> {
    using v2 = __nv_bfloat162;
    static __device__ __forceinline__ float2 to_f2(uint32_t u) {
        // bf16 -> fp32 is a 16-bit shift
        float2 r;
        r.x = __uint_as_float(u << 16);
        r.y = __uint_as_float(u & 0xFFFF0000u);
        return r;
    }
    static __device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
    static __device__ __forceinline__ __nv_bfloat16 from_float(float x) { return __float2bfloat16_rn(x); }
};

// Programmatic dependent launch inside one call (the kernels of a compress follow one another on one
// stream): a kernel lets its successor be scheduled as soon as every CTA has started (or exited), so the
// successor's CTAs take over the SMs as they become free and run whatever does not depend on the
// predecessor; before the first access that does, they wait for the predecessor to be complete and
// its writes to be visible.  Both instructions do nothing in a launch without the attribute.
__device__ __forceinline__ void kvr_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }
__device__ __forceinline__ void kvr_pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }

// element-wise middle of three
__device__ __forceinline__ float kvr_med3(float x, float y, float z) {
    return fmaxf(fminf(x, y), fminf(fmaxf(x, y), z));
}
// what Algorithm 2 makes of a token's three collected numbers: their middle (the paper), or their mean
__device__ __forceinline__ float kvr_comb3(float x, float y, float z, int mean) {
    return mean ? (x + y + z) * (1.0f / 3.0f) : kvr_med3(x, y, z);
}
// Launch `kern` on `st`; dependent = true: as a programmatic dependent of the kernel launched before it
// on that stream (see kvr_pdl_trigger / kvr_pdl_wait: the kernel must wait before it touches anything
// its predecessor writes).
template <typename... KArgs, typename... Args>
inline cudaError_t kvr_launch_after(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    bool dependent, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}
#endif
