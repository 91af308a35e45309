// Internal declarations shared by the kernel files and the host layer of libhivis.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/hivis.h"

typedef __nv_bfloat16 bf16;
typedef unsigned long long u64;

#define HIVIS_MAX_DEVICES 64   // per-device caches of function attributes are indexed by device ordinal

// ---------------------------------------------------------------------------------------------
// Skinny linear layer  out[b][n] = sum_k W[n][k] * x[b][k]  with a fused input stage (PRO_*)
// and a fused output stage (EPI_*).  Two kernel families share these arguments:
//   gemv_alu : fp32 FMAs, one batch row per CTA column (B == 1, or fp32 weights)
//   gemm_mma : bf16 tensor-core tiles, up to 16 batch rows per pass
// ---------------------------------------------------------------------------------------------
enum { PRO_PLAIN = 0, PRO_NORM = 1, PRO_FUSE = 2 };
enum { EPI_FUSE = 0, EPI_QKV = 1, EPI_OPROJ = 2, EPI_GATEUP = 3, EPI_DOWN = 4, EPI_LM = 5 };

struct LinArgs {
    const void* W;        // [N][K] in the context dtype
    int N, K, B;
    int ldb;              // row stride (elements) of the ssq buffers = batch capacity
    // ---- input stage
    const float* xin;     // PRO_PLAIN / PRO_NORM (alu): [B][K] fp32
    const bf16* xin_h;    // mma: [B][K] bf16 (already multiplied by the norm gain where one applies)
    const void* gamma;    // PRO_NORM (alu): [K] gain, context dtype
    float eps;
    const float* feat;    // PRO_FUSE (alu): [B][d] fp32 hidden feature
    const void* feat_h;   // PRO_FUSE (mma): [B][d] bf16 hidden feature
    const void* embed;    // PRO_FUSE: [vocab][d], context dtype
    const int* ids;       // PRO_FUSE: token of row b = ids[b * id_stride]; if null, decoded from keys
    int id_stride;
    const u64* keys;      // PRO_FUSE: packed argmax keys, row b at keys[b * key_stride]
    int key_stride;
    int d;
    int vocab;            // PRO_FUSE: ids outside [0, vocab) are read as token 0 and raise *id_flag
    int* id_flag;
    // ---- scale recovered from per-tile partial sums of squares (mma EPI_QKV / EPI_GATEUP):
    //      s[b] = rsqrt( sum_t ssq_in[t*ldb + b] / K + eps )
    const float* ssq_in;
    int ssq_tiles;
    // ---- output stage
    const void* bias;     // EPI_QKV: [N] context dtype, nullable
    const float* rho;     // EPI_FUSE: [N] fp32 residual row, nullable
    const float* addend;  // EPI_OPROJ (u), EPI_DOWN (y): [B][N] fp32
    float* out;           // fp32 result [B][N] (EPI_GATEUP: [B][N/2]); nullable
    bf16* out_h;          // bf16 copy [B][N] (EPI_GATEUP: [B][N/2]); nullable
    const void* gamma_out;// EPI_FUSE / EPI_OPROJ: out_h = bf16(gamma_out[n] * value), context dtype
    float* ssq_out;       // EPI_FUSE / EPI_OPROJ (mma): [tiles][ldb] partial sums of squares
    u64* keys_out;        // EPI_LM: row b at keys_out[b * keys_out_stride]
    int keys_out_stride;
    float* logits_out;    // EPI_LM: nullable, row b at logits_out[b * logits_ld]
    long long logits_ld;
};

// Rows of W covered by one CTA of the tensor-core kernel.
#define HIVIS_MMA_TILE_ROWS 32

cudaError_t launch_gemv_alu(int dtype, int pro, int epi, const LinArgs& a, cudaStream_t st);
cudaError_t launch_gemm_mma(int pro, int epi, const LinArgs& a, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Decode attention over the text-only cache (one new position per sequence).
// ---------------------------------------------------------------------------------------------
struct AttnArgs {
    const float* qkv;     // [B][ld]: q | k | v of the new position, before RoPE
    int ld;
    void* Kc;             // [slot][Hkv][max_len][dh], context dtype, K stored after RoPE
    void* Vc;
    const int* slots;     // [B]
    const int* pos0;      // [B] cache row of draft step 0
    int step;             // this step's row = pos0[b] + step
    const double* inv_freq;   // [dh/2]  base^(-2i/dh)
    int Hq, Hkv, dh, max_len, B;
    float scale;          // 1/sqrt(dh)
    int chunk;            // cache rows per split
    int nsplit;           // grid.x
    float* part_acc;      // [B][Hq][nsplit][dh]
    float* part_ml;       // [B][Hq][nsplit][2]
    int* counters;        // [B][Hq] arrival counters, zero between launches
    float* attn;          // [B][Hq*dh] fp32
    bf16* attn_h;         // [B][Hq*dh] bf16 copy
    int lo_rows;          // > 0: rounding remainders of attn_h go to rows b + lo_rows
};
cudaError_t launch_attention(int dtype, const AttnArgs& a, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Persistent chain kernel (one sequence, all k steps in one cooperative launch).
// ---------------------------------------------------------------------------------------------
enum { PH_FC = 0, PH_QKV, PH_O, PH_GU, PH_DOWN, PH_LM, PH_COUNT };

struct ChainPhase {
    const void* W;        // [N][K], context dtype
    int N, K;
};

struct ChainArgs {
    ChainPhase ph[PH_COUNT];
    int k;
    int d, qw, kvw, F, V, Hq, Hkv, dh, max_len;
    float eps, scale;
    const void *norm1, *norm2, *bqkv, *embed;
    const float* rho;          // [n_resid][d] fp32, nullable
    int n_resid;
    int slot;
    int* kv_len;
    const float* pend_feat;    // [slots][d]
    const int* pend_id;
    float *u, *qkv, *attn, *y, *act, *feat;
    u64* keys;                 // [k]
    const int* forced;         // [k], nullable
    float* logits_out;         // [k][V], nullable
    const float* gumbel_u;     // [k][V] uniform numbers in (0, 1), nullable: the token is drawn, not the maximum
    float inv_t;               // 1 / temperature of the draw
    int32_t* out_ids;          // [k]
    void *Kc, *Vc;
    const double* inv_freq;
    float *part_acc, *part_ml;
    int* counters;
    int attn_chunk, attn_nsplit;
    u64* bar_counter;          // arrival counter of the grid barrier, only ever incremented
    u64 bar_base;              // its value when this launch starts
    long long wait_cycles;     // limit of every device-side wait, in SM clock cycles
    int* error_flag;           // set non-zero by a kernel that gave up on a wait
    int* id_flag;              // set non-zero when a token id outside [0, V) reached the embedding lookup
    int off_x, off_part, off_bar, off_misc;   // shared-memory layout, filled by the launcher
};
// shared memory the kernel needs for these dimensions on `grid` CTAs; 0 = does not fit
size_t chain_smem_bytes(const ChainArgs& a, int dtype, int grid);
cudaError_t launch_draft_chain(ChainArgs& a, int dtype, int grid, cudaStream_t st);
int chain_barriers_per_step();

struct SlotList {
    int n;
    int slot[HIVIS_MAX_BATCH];
};
struct CuSeqlens {
    int v[HIVIS_MAX_BATCH + 1];
};

// ---------------------------------------------------------------------------------------------
// Tensor-core chain kernel (bf16 weights, 1..16 sequences): all k steps in one cooperative launch,
// weights streamed by TMA into a shared-memory ring, tcgen05.mma with the weights as the M operand
// (128 rows) and the batch as N (16 columns), accumulators in tensor memory.
// ---------------------------------------------------------------------------------------------
#define TC_OP_ROWS 32          // rows of every bf16 operand buffer that the tensor maps cover
enum { TCM_W = 0,              // PH_COUNT weight maps, box 64 x 128
       TCM_X_FEAT = PH_COUNT, TCM_X_XQ, TCM_X_ATTN, TCM_X_XM, TCM_X_ACT,   // operand maps, box 64 x 16
       TCM_X_EMB,              // gathered embedding rows, box 64 x 16
       TCM_K, TCM_V,           // the caches, box 64 x 32 rows
       TCM_COUNT };
struct TcMaps {
    alignas(64) unsigned char m[TCM_COUNT][128];     // CUtensorMap objects
};
struct TcArgs {
    ChainPhase ph[PH_COUNT];
    int k, B;
    int lo;                    // > 0: operand rows [lo, lo + B) carry the bf16 rounding remainders of rows [0, B)
    int d, qw, kvw, F, V, Hq, Hkv, dh, max_len;
    float eps, scale;
    const bf16 *norm1, *norm2, *bqkv;
    const float* rho;          // [n_resid][d] fp32, nullable
    int n_resid;
    const int *slots, *pos0, *cur_id;     // [B]
    const int* forced;         // [B][k], nullable
    u64* keys;                 // [B][key_stride]
    int key_stride;
    float *u, *qkv, *attn, *y, *feat;     // fp32 activations [B][width]
    bf16 *feat_h, *xq_h, *attn_h, *xm_h, *act_h;   // bf16 operands [TC_OP_ROWS][width]
    bf16* xe_h;                // [TC_OP_ROWS][d] embedding rows of the step's tokens (the set-up kernel zeroes rows >= B)
    const bf16* embed;         // [V][d]
    float *ssq1, *ssq2;        // [tiles*4][16] partial sums of squares of u / y
    float* logits_out;         // [B][k][V], nullable
    const float* gumbel_u;     // [B][k][V] uniform numbers in (0, 1), nullable: tokens are drawn, not the maximum
    float inv_t;               // 1 / temperature of the draw
    float* partial;            // [grid*2][16][128] split-tile partial accumulators
    int* tile_ctr;             // arrival counters of split tiles, zero between phases
    void *Kc, *Vc;
    const double* inv_freq;
    float2* rope_tab;          // [2][16][dh/2] (cos, sin) per sequence at the current step, halves alternate
    float *part_acc, *part_ml;
    int* counters;
    int attn_nslot;            // partial slots per (sequence, head): >= 32-row blocks of the longest sequence
    u64* bar_counter;
    u64 bar_base;
    long long wait_cycles;     // limit of every device-side wait, in SM clock cycles
    int* error_flag;
    int* id_flag;              // set non-zero when a token id outside [0, V) reached the embedding lookup
    u64* phase_t;              // nullable: [k][HIVIS_PHASE_EVENTS][grid] time stamps (HIVIS_OPT_PHASE_TIMES)
    int l2_keep;               // bit p set: the weights of phase p are loaded with the keep-in-L2 policy
    // The grid barriers of a step are numbered 0 gather, 1 FC, 2 QKV, 3 attention, 4 O, 5 gate/up, 6 down, 7 LM head.
    // A launch runs the part [seq_first, seq_last] of every step (0..7: the whole step); what lies outside does no work
    // and arrives nowhere, and bar_base is set as if the barriers before seq_first had been completed already.
    int seq_first, seq_last;
};
// fills `maps` for the given buffers; returns cudaSuccess or an error (driver entry point missing, bad shape)
cudaError_t tc_build_maps(TcMaps* maps, const ChainPhase* ph, int d, int qw, int F, const bf16* feat_h,
                          const bf16* xq_h, const bf16* attn_h, const bf16* xm_h, const bf16* act_h, const bf16* xe_h,
                          const void* Kc, const void* Vc, long long cache_rows, int dh);
bool tc_supported(int d, int dh, int Hq, int Hkv, int F);
int tc_max_tiles(const ChainPhase* ph);
cudaError_t launch_tc_chain(const TcMaps& maps, const TcArgs& a, int grid, cudaStream_t st);
cudaError_t launch_tc_setup(const SlotList& sl, int k, int d, int lo, int* d_slots, int* d_pos0, int* kv_len,
                            const float* pend_feat, const int* pend_id, float* feat, bf16* feat_h,
                            int* cur_id, u64* keys, int key_stride, const bf16* embed, int vocab, bf16* xe_h,
                            int* id_flag, cudaStream_t st);
int tc_barriers_per_step();
int tc_lo_offset(int B);

// ---------------------------------------------------------------------------------------------
// Prefix build on the tensor cores (kernels_prefill_tc.cu): two tcgen05 GEMMs over all packed pairs.
// ---------------------------------------------------------------------------------------------
struct PrefillTcArgs {
    int n_pairs, pair_cap;     // packed pairs of the call; capacity of the pair-major buffers
    int d, kvw, Hkv, dh, max_len, vocab;
    float eps;
    const int32_t* ids;        // [n_pairs]
    const bf16* hidden;        // [n_pairs][d] the caller's hidden states
    const bf16 *embed, *fc, *wkv, *bkv, *norm1;      // wkv: rows [K ; V] of the stacked QKV matrix, bkv nullable
    const float* rho0;         // [d] nullable
    bf16 *xe, *xq;             // [pair_cap][d] gathered embedding rows; gamma_1 * u
    float* ssq;                // [ceil(d / 128)][pair_cap]
    float2* rope;              // [pair_cap][dh / 2] scratch: (cos, sin) at every pair's position
    const int *slot_of, *row_of;
    const double* inv_freq;
    bf16 *Kc, *Vc;
    long long wait_cycles;
    int *error_flag, *id_flag;
};
bool prefill_tc_supported(int d, int kvw);
cudaError_t launch_prefill_tc(const PrefillTcArgs& a, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Tree drafting (kernels_tree.cu): device-side bookkeeping of one draft tree.
// ---------------------------------------------------------------------------------------------
#define TREE_MAX_TOPK HIVIS_TREE_MAX_TOPK
#define TREE_MAX_DEPTH HIVIS_MAX_K
#define TREE_MAX_CAND (TREE_MAX_TOPK + (TREE_MAX_DEPTH - 1) * TREE_MAX_TOPK * TREE_MAX_TOPK)
struct TreeBufs {
    int* P;                    // [1] rows the slot held when the tree was drafted (row P = the root position)
    // the frontier of the level being run: candidate index (-1: the root), token, cumulative log-probability, row of
    // the previous level's output that feeds it, tree row (offset from P), tree rows of its ancestors (root first)
    int *fr_cand, *fr_tok, *fr_pslot, *fr_store, *fr_anc;      // [TOPK], ..., [TOPK][DEPTH]
    float* fr_score;
    int* top_tok;              // [TOPK][TOPK] the top-k tokens of every frontier node's distribution
    float* top_lp;             //              and their log-probabilities
    // every candidate ever proposed, in creation order
    int *cand_n, *cand_tok, *cand_par, *cand_depth, *cand_store, *cand_keep, *cand_pos;
    float* cand_score;
    // the kept nodes (the draft tree handed to the caller), for the verification
    int *kept_n, *kept_tok, *kept_par, *kept_store;
    u64* row_keys;             // [keep + 1] argmax keys of the target's rows
    // top-k of a level's logits: per node and 4096-logit piece the (max, sum exp) and the piece's largest keys
    float2* piece_stats;       // [TOPK][pieces]
    u64* piece_keys;           // [TOPK][pieces][TOPK]
};
int tree_topk_pieces(int V);
cudaError_t launch_tree_begin(int slot, int d, const int* kv_len, const float* pend_feat, const int* pend_id, float* feat,
                              bf16* feat_h, int* cur_id, int* d_slots, const TreeBufs& T, cudaStream_t st);
cudaError_t launch_tree_gather(int nb, int d, const float* g_prev, const TreeBufs& T, float* feat, bf16* feat_h, int* cur_id,
                               cudaStream_t st);
cudaError_t launch_tree_attention(int dtype, int nb, const float* qkv, int ld, int Hq, int Hkv, int dh, int max_len,
                                  int slot, int level, const TreeBufs& T, const double* inv_freq, void* Kc, void* Vc,
                                  float* attn, bf16* attn_h, int lo_rows, cudaStream_t st);
// the level's rows as the tensor-core chain kernel reads them (`rows` = all operand rows, so that those beyond the
// level are cleared; g_prev non-null: the rows are gathered from the previous level's outputs on the way)
cudaError_t launch_tree_operands_tc(int nb, int rows, int d, int lo_rows, const float* feat, const int* cur_id,
                                    const float* g_prev, const TreeBufs& T, const bf16* embed, int vocab, bf16* feat_h,
                                    bf16* xe_h, int* pos0, int* id_flag, cudaStream_t st);
cudaError_t launch_tree_topk(int nb, const float* logits, int V, int topk, const TreeBufs& T, cudaStream_t st);
cudaError_t launch_tree_select(int level, int depth, int nb, int topk, const TreeBufs& T, cudaStream_t st);
cudaError_t launch_tree_finalize(int keep, const TreeBufs& T, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                                 int32_t* out_count, cudaStream_t st);
cudaError_t launch_tree_verify(int dtype, int logits_dtype, int slot, int depth, int rows, int V, int Hkv, int dh, int max_len,
                               const TreeBufs& T, const void* logits, void* Kc, void* Vc, int* kv_len, int32_t* out_accept,
                               int32_t* out_path, int32_t* out_next, int32_t* out_kv_len, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// Small kernels: state set-up, prefill bookkeeping, verification, layout changes, taps.
// ---------------------------------------------------------------------------------------------

// draft set-up: slots -> device, pos0 = kv_len[slot], feat = pending feature, ids = pending id;
// clears the argmax keys [B][k]; advances kv_len by k.
cudaError_t launch_draft_setup(const SlotList& sl, int k, int d, int* d_slots, int* d_pos0,
                               int* kv_len, const float* pend_feat, const int* pend_id, float* feat,
                               bf16* feat_h, int* cur_id, u64* keys, int key_stride, cudaStream_t st);
// decode keys [B][k] into out_ids [B][k]
cudaError_t launch_draft_finish(int B, int k, const u64* keys, int key_stride, int32_t* out_ids,
                                cudaStream_t st);

// residual rows (context dtype) -> fp32 rho [R][d] (no projection)
cudaError_t launch_convert_rows(int dtype, const void* src, float* dst, long long n, cudaStream_t st);
cudaError_t launch_f32_to_bf16(const float* src, bf16* dst, long long n, cudaStream_t st);
cudaError_t launch_bf16_to_f32(const bf16* src, float* dst, long long n, cudaStream_t st);

// prefill bookkeeping: for every packed entry j: slot_of[j], row_of[j] (-1 for the pending pair);
// stores the pending pair; updates kv_len.
cudaError_t launch_prefill_setup(int dtype, const SlotList& sl, const CuSeqlens& cu,
                                 const SlotList& start /* -1 = append */, int d, const int32_t* ids,
                                 const void* hidden, int* kv_len, float* pend_feat, int* pend_id,
                                 int* slot_of, int* row_of, cudaStream_t st);
// RoPE(K) and store K,V rows of a chunk of packed entries
cudaError_t launch_kv_append(int dtype, const float* kv /*[P][2*kvw]*/, int P, const int* slot_of,
                             const int* row_of, const double* inv_freq, int Hkv, int dh, int max_len,
                             void* Kc, void* Vc, cudaStream_t st);

// verification in one launch: row argmax over [B][k+1][V], accept length / next token / rollback.
// keys [B][k+1] and arrivals [B] must be zero on entry and are left zero.
cudaError_t launch_verify(int logits_dtype, const SlotList& sl, int k, int V, const int32_t* draft_ids,
                          const void* logits, u64* keys, int* arrivals, int* kv_len, int32_t* out_accept,
                          int32_t* out_next, int32_t* out_kv_len, cudaStream_t st, int* n_launches);

// verification by speculative sampling: per-row softmax statistics, then acceptance tests, the draw of the next token
// and the rollback; stats: scratch of sampled_stats_entries(max_batch, max_k, V) entries (one per piece of a row)
int sampled_stats_entries(int max_batch, int max_k, int V);
cudaError_t launch_verify_sampled(int logits_dtype, const SlotList& sl, int k, int V, float temperature,
                                  const int32_t* draft_ids, const float* draft_logits, const void* target_logits,
                                  float2* stats, const float* u_accept, const float* u_sample, int* kv_len,
                                  int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len, cudaStream_t st);

cudaError_t launch_set_int(int* p, int v, cudaStream_t st);
// kv_len[sl.slot[b]] = rows.v[b] for b < sl.n
cudaError_t launch_set_rows(const SlotList& sl, const CuSeqlens& rows, int* kv_len, cudaStream_t st);

// weight re-layout at init
cudaError_t launch_copy_rows(const void* src, void* dst, long long rows, long long row_bytes,
                             long long dst_row0, long long dst_row_step, cudaStream_t st);

cudaError_t launch_read_kv(int dtype, const void* Kc, const void* Vc, int slot, int row0, int n,
                           int Hkv, int dh, int max_len, float* out_k, float* out_v, cudaStream_t st);

// ---------------------------------------------------------------------------------------------
// device helpers
// ---------------------------------------------------------------------------------------------
#ifdef __CUDACC__
// Order-preserving map of a float to 32 bits (NaN -> 0 so that it never wins), packed with the
// index so that a 64-bit integer max picks the largest value and, among equals, the lowest index.
__device__ __forceinline__ u64 pack_key(float v, int idx) {
    unsigned int u = __float_as_uint(v);
    u = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    if (v != v) u = 0u;
    return ((u64)u << 32) | (u64)(0xFFFFFFFFu - (unsigned int)idx);
}
// the value whose maximum is the drawn token: logit / T plus standard Gumbel noise made from a uniform number
__device__ __forceinline__ float gumbel_perturbed(float logit, float inv_t, float u) {
    return fmaf(logit, inv_t, -logf(-logf(u)));
}
__device__ __forceinline__ int key_index(u64 key) {
    return (int)(0xFFFFFFFFu - (unsigned int)(key & 0xFFFFFFFFull));
}
// A token id on its way to the embedding table: an id outside [0, vocab) is read as token 0 and recorded in
// *id_flag (reported by hivis_status), so that no lookup leaves the table whatever sits in device memory.
__device__ __forceinline__ int checked_token(int id, int vocab, int* id_flag) {
    if (id >= 0 && id < vocab) return id;
    if (id_flag) *(volatile int*)id_flag = 1;
    return 0;
}
__device__ __forceinline__ float bf16_lo(unsigned int w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(unsigned int w) { return __uint_as_float(w & 0xFFFF0000u); }

template <typename WT>
__device__ __forceinline__ float load_as_float(const void* p, long long i);
template <>
__device__ __forceinline__ float load_as_float<float>(const void* p, long long i) {
    return ((const float*)p)[i];
}
template <>
__device__ __forceinline__ float load_as_float<bf16>(const void* p, long long i) {
    return __bfloat162float(((const bf16*)p)[i]);
}
template <typename WT>
__device__ __forceinline__ void store_from_float(void* p, long long i, float v);
template <>
__device__ __forceinline__ void store_from_float<float>(void* p, long long i, float v) {
    ((float*)p)[i] = v;
}
template <>
__device__ __forceinline__ void store_from_float<bf16>(void* p, long long i, float v) {
    ((bf16*)p)[i] = __float2bfloat16_rn(v);
}

// 16-byte streaming load of weights: read-only path, do not keep in L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
// 16-byte load of an activation written by an earlier kernel: L2 only.
__device__ __forceinline__ uint4 ld_act(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.cg.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
#endif
