// Tree drafting and greedy tree verification: the kernels around the layer.
//
// A draft tree is built level by level.  Level 0 runs the pending pair (one row); level l >= 1 runs the `topk`
// frontier nodes of depth l as a batch of rows through the same fused linear kernels as a chained step.  What is
// specific to the tree lives here: the gather of every node's input (the layer output of the forward that proposed
// it, its token), tree attention (a node sees the prefix, its ancestors and itself), log-softmax + top-k of every
// node's logits, the choice of the next frontier by cumulative log-probability, the final ranking of all
// candidates, and - after the target has scored the kept nodes - the walk along the accepted path with the
// compaction of its K/V rows.  All bookkeeping stays on the device; the host only sequences launches.
//
// Where the rows of the tree live: the node that is the j-th of the level-l frontier keeps its K/V row in cache row
// P + 1 + (l - 1) * topk + j of its slot (P = rows of the slot before the draft, row P = the root position).
#include "attn_body.cuh"

// ------------------------------------------------------------------------------------------ begin / gather
__global__ void tree_begin_kernel(int slot, int d, const int* kv_len, const float* pend_feat, const int* pend_id,
                                  float* feat, bf16* feat_h, int* cur_id, int* d_slots, TreeBufs T) {
    if (threadIdx.x == 0) {
        *T.P = kv_len[slot];
        *T.cand_n = 0;
        cur_id[0] = pend_id[slot];
        T.fr_cand[0] = -1;
        T.fr_store[0] = 0;
        T.fr_score[0] = 0.f;
    }
    if (threadIdx.x < TREE_MAX_TOPK) d_slots[threadIdx.x] = slot;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = pend_feat[(long long)slot * d + i];
        feat[i] = v;
        feat_h[i] = __float2bfloat16_rn(v);
    }
}
cudaError_t launch_tree_begin(int slot, int d, const int* kv_len, const float* pend_feat, const int* pend_id, float* feat,
                              bf16* feat_h, int* cur_id, int* d_slots, const TreeBufs& T, cudaStream_t st) {
    tree_begin_kernel<<<1, 256, 0, st>>>(slot, d, kv_len, pend_feat, pend_id, feat, feat_h, cur_id, d_slots, T);
    return cudaGetLastError();
}

// row j of the level's input: the layer output of the forward that proposed node j, and node j's token
__global__ void tree_gather_kernel(int d, const float* g_prev, TreeBufs T, float* feat, bf16* feat_h, int* cur_id) {
    const int j = blockIdx.x;
    const float* src = g_prev + (long long)T.fr_pslot[j] * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = src[i];
        feat[(long long)j * d + i] = v;
        feat_h[(long long)j * d + i] = __float2bfloat16_rn(v);
    }
    if (threadIdx.x == 0) cur_id[j] = T.fr_tok[j];
}
cudaError_t launch_tree_gather(int nb, int d, const float* g_prev, const TreeBufs& T, float* feat, bf16* feat_h, int* cur_id,
                               cudaStream_t st) {
    tree_gather_kernel<<<nb, 256, 0, st>>>(d, g_prev, T, feat, feat_h, cur_id);
    return cudaGetLastError();
}

// The level's rows in the form the tensor-core chain kernel reads them: the features as bf16 rows with their rounding
// remainders `lo_rows` rows further down, the embedding rows of the nodes' tokens (zero rows beyond the level: the
// tiled copy always brings all rows), and a row count of zero per column (the kernel's own attention is not used).
// With g_prev the rows are gathered on the way (row j = the layer output of the forward that proposed node j, and node j's
// token); without, they are taken from feat / cur_id as tree_begin left them.
__global__ void tree_operands_tc_kernel(int nb, int d, int lo_rows, const float* feat, const int* cur_id, const float* g_prev,
                                        TreeBufs T, const bf16* embed, int vocab, bf16* feat_h, bf16* xe_h, int* pos0,
                                        int* id_flag) {
    const int j = blockIdx.x;
    if (j >= nb) {
        for (int i = threadIdx.x; i < (d >> 3); i += blockDim.x)
            ((uint4*)(xe_h + (long long)j * d))[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    if (threadIdx.x == 0) pos0[j] = 0;
    const float* src = g_prev ? g_prev + (long long)T.fr_pslot[j] * d : feat + (long long)j * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = src[i];
        const bf16 hi = __float2bfloat16_rn(v);
        feat_h[(long long)j * d + i] = hi;
        feat_h[(long long)(j + lo_rows) * d + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    const int id = checked_token(g_prev ? T.fr_tok[j] : cur_id[j], vocab, id_flag);
    for (int i = threadIdx.x; i < (d >> 3); i += blockDim.x)
        ((uint4*)(xe_h + (long long)j * d))[i] = ((const uint4*)(embed + (long long)id * d))[i];
}
cudaError_t launch_tree_operands_tc(int nb, int rows, int d, int lo_rows, const float* feat, const int* cur_id,
                                    const float* g_prev, const TreeBufs& T, const bf16* embed, int vocab, bf16* feat_h,
                                    bf16* xe_h, int* pos0, int* id_flag, cudaStream_t st) {
    tree_operands_tc_kernel<<<rows, 256, 0, st>>>(nb, d, lo_rows, feat, cur_id, g_prev, T, embed, vocab, feat_h, xe_h, pos0,
                                                  id_flag);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ K/V rows of the level
template <typename WT>
__global__ void tree_kv_write_kernel(const float* qkv, int ld, int qw, int Hkv, int dh, int max_len, int slot, int level,
                                     TreeBufs T, const double* inv_freq, void* Kc, void* Vc) {
    __shared__ float2 s_cs[128];                        // (cos, sin) of the level's position: the same for every head
    const int j = blockIdx.x;
    const int P = *T.P;
    const int row = P + T.fr_store[j], pos = P + level;
    const int half = dh / 2, kvw = Hkv * dh;
    for (int e = threadIdx.x; e < half; e += blockDim.x) {
        float c, s;
        rope_cs(pos, inv_freq[e], c, s);
        s_cs[e] = make_float2(c, s);
    }
    __syncthreads();
    const float* k = qkv + (long long)j * ld + qw;
    const float* v = k + kvw;
    for (int i = threadIdx.x; i < Hkv * half; i += blockDim.x) {
        const int h = i / half, e = i % half;
        const float c = s_cs[e].x, s = s_cs[e].y;
        const float x0 = k[h * dh + e], x1 = k[h * dh + e + half];
        const long long o = (((long long)slot * Hkv + h) * max_len + row) * dh;
        store_from_float<WT>(Kc, o + e, x0 * c - x1 * s);
        store_from_float<WT>(Kc, o + e + half, x1 * c + x0 * s);
    }
    for (int i = threadIdx.x; i < kvw; i += blockDim.x) {
        const int h = i / dh, e = i % dh;
        const long long o = (((long long)slot * Hkv + h) * max_len + row) * dh;
        store_from_float<WT>(Vc, o + e, v[i]);
    }
}

// ------------------------------------------------------------------------------------------ tree attention
// One CTA of four warps per (query head, node).  The node attends to the prefix rows [0, P), to the rows of its
// ancestors (the root position first) and to its own row: `level` + 1 tree rows.  Blocks of 32 rows are dealt to the
// warps in turn.  Scores: a lane takes one row of the block and the whole dot product with the query (in shared
// memory), so no shuffle is needed; the block's probabilities then go through an online softmax, and for the weighted
// sum of the V rows a lane owns DH/32 output elements and every row's probability is broadcast from its lane.  The four
// warps' (max, sum, accumulator) are merged at the end.
template <typename WT, int DH>
__device__ __forceinline__ float tree_row_dot(const void* Kc, long long o, const float* q) {
    float sc = 0.f;
    if constexpr (sizeof(WT) == 2) {
        const uint4* kp = (const uint4*)((const bf16*)Kc + o);
#pragma unroll
        for (int c = 0; c < DH / 8; ++c) {
            const uint4 w = __ldg(kp + c);
            sc = fmaf(q[8 * c + 0], bf16_lo(w.x), sc); sc = fmaf(q[8 * c + 1], bf16_hi(w.x), sc);
            sc = fmaf(q[8 * c + 2], bf16_lo(w.y), sc); sc = fmaf(q[8 * c + 3], bf16_hi(w.y), sc);
            sc = fmaf(q[8 * c + 4], bf16_lo(w.z), sc); sc = fmaf(q[8 * c + 5], bf16_hi(w.z), sc);
            sc = fmaf(q[8 * c + 6], bf16_lo(w.w), sc); sc = fmaf(q[8 * c + 7], bf16_hi(w.w), sc);
        }
    } else {
        const float4* kp = (const float4*)((const float*)Kc + o);
#pragma unroll
        for (int c = 0; c < DH / 4; ++c) {
            const float4 w = __ldg(kp + c);
            sc = fmaf(q[4 * c + 0], w.x, sc); sc = fmaf(q[4 * c + 1], w.y, sc);
            sc = fmaf(q[4 * c + 2], w.z, sc); sc = fmaf(q[4 * c + 3], w.w, sc);
        }
    }
    return sc;
}
template <typename WT, int DH>
__global__ void __launch_bounds__(128) tree_attn_kernel(const float* qkv, int ld, int Hq, int Hkv, int max_len, int slot,
                                                        int level, TreeBufs T, const double* inv_freq, float scale,
                                                        const void* Kc, const void* Vc, float* attn, bf16* attn_h,
                                                        int lo_rows) {
    constexpr int EPL = DH / 32;
    __shared__ float s_m[4], s_l[4], s_acc[4][DH];
    __shared__ __align__(16) float s_q[DH];
    __shared__ float2 s_cs[DH / 2];
    const int h = blockIdx.x, j = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int P = *T.P, pos = P + level, kvh = h / (Hq / Hkv), half = DH / 2;
    if (threadIdx.x < half) {
        float c, s;
        rope_cs(pos, inv_freq[threadIdx.x], c, s);
        s_cs[threadIdx.x] = make_float2(c, s);
    }
    __syncthreads();
    // the rotated, scaled query
    const float* qh = qkv + (long long)j * ld + h * DH;
    for (int i = threadIdx.x; i < DH; i += 128) {
        const int f = i % half;
        const float c = s_cs[f].x, s = s_cs[f].y;
        const float x = qh[i], y = qh[i < half ? i + half : i - half];
        s_q[i] = (i < half ? x * c - y * s : x * c + y * s) * scale;
    }
    __syncthreads();
    const long long base = ((long long)slot * Hkv + kvh) * max_len;
    const int nrows = P + level + 1;
    float m = -INFINITY, l = 0.f, acc[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
    for (int r0 = warp * 32; r0 < nrows; r0 += 128) {
        const int r = r0 + lane;
        const bool ok = r < nrows;
        int row = ok ? r : 0;
        if (ok && r >= P) {
            const int a = r - P;                                     // a-th tree row on the path: ancestors, then the node
            row = P + (a < level ? T.fr_anc[j * TREE_MAX_DEPTH + a] : T.fr_store[j]);
        }
        const float sc = ok ? tree_row_dot<WT, DH>(Kc, (base + row) * DH, s_q) : -INFINITY;
        float bm = sc;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, off));
        const float mn = fmaxf(m, bm);                               // finite: the block has at least one row
        const float corr = expf(m - mn), p = ok ? expf(sc - mn) : 0.f;
        float ps = p;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, off);
        l = l * corr + ps;
        m = mn;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[e] *= corr;
        const int nr = min(32, nrows - r0);
#pragma unroll 4
        for (int t = 0; t < nr; ++t) {
            const float pj = __shfl_sync(0xffffffffu, p, t);
            const int rowj = __shfl_sync(0xffffffffu, row, t);
            const long long o = (base + rowj) * DH + lane * EPL;
            if constexpr (sizeof(WT) == 2 && EPL == 4) {
                const uint2 w = __ldg((const uint2*)((const bf16*)Vc + o));
                acc[0] = fmaf(pj, bf16_lo(w.x), acc[0]); acc[1] = fmaf(pj, bf16_hi(w.x), acc[1]);
                acc[2] = fmaf(pj, bf16_lo(w.y), acc[2]); acc[3] = fmaf(pj, bf16_hi(w.y), acc[3]);
            } else if constexpr (sizeof(WT) == 2 && EPL == 2) {
                const unsigned w = __ldg((const unsigned*)((const bf16*)Vc + o));
                acc[0] = fmaf(pj, bf16_lo(w), acc[0]); acc[1] = fmaf(pj, bf16_hi(w), acc[1]);
            } else {
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[e] = fmaf(pj, load_as_float<WT>(Vc, o + e), acc[e]);
            }
        }
    }
    if (lane == 0) { s_m[warp] = m; s_l[warp] = l; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) s_acc[warp][lane * EPL + e] = acc[e];
    __syncthreads();
    if (warp == 0) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, s_m[w]);
        float L = 0.f, A[EPL];
#pragma unroll
        for (int e = 0; e < EPL; ++e) A[e] = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float f = s_l[w] > 0.f ? expf(s_m[w] - M) : 0.f;   // a warp without rows contributes nothing
            L += s_l[w] * f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) A[e] += s_acc[w][lane * EPL + e] * f;
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) {
            const float o = A[e] / L;
            const long long oi = (long long)j * Hq * DH + h * DH + lane * EPL + e;
            attn[oi] = o;
            const bf16 hi = __float2bfloat16_rn(o);
            attn_h[oi] = hi;
            if (lo_rows > 0) attn_h[oi + (long long)lo_rows * Hq * DH] = __float2bfloat16_rn(o - __bfloat162float(hi));
        }
    }
}

cudaError_t launch_tree_attention(int dtype, int nb, const float* qkv, int ld, int Hq, int Hkv, int dh, int max_len,
                                  int slot, int level, const TreeBufs& T, const double* inv_freq, void* Kc, void* Vc,
                                  float* attn, bf16* attn_h, int lo_rows, cudaStream_t st) {
    const int qw = Hq * dh;
    const float scale = 1.0f / sqrtf((float)dh);
    if (dtype == HIVIS_BF16)
        tree_kv_write_kernel<bf16><<<nb, 256, 0, st>>>(qkv, ld, qw, Hkv, dh, max_len, slot, level, T, inv_freq, Kc, Vc);
    else
        tree_kv_write_kernel<float><<<nb, 256, 0, st>>>(qkv, ld, qw, Hkv, dh, max_len, slot, level, T, inv_freq, Kc, Vc);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)Hq, (unsigned)nb);
    if (dtype == HIVIS_BF16) {
        if (dh == 128) tree_attn_kernel<bf16, 128><<<grid, 128, 0, st>>>(qkv, ld, Hq, Hkv, max_len, slot, level, T, inv_freq, scale, Kc, Vc, attn, attn_h, lo_rows);
        else tree_attn_kernel<bf16, 64><<<grid, 128, 0, st>>>(qkv, ld, Hq, Hkv, max_len, slot, level, T, inv_freq, scale, Kc, Vc, attn, attn_h, lo_rows);
    } else {
        if (dh == 128) tree_attn_kernel<float, 128><<<grid, 128, 0, st>>>(qkv, ld, Hq, Hkv, max_len, slot, level, T, inv_freq, scale, Kc, Vc, attn, attn_h, lo_rows);
        else tree_attn_kernel<float, 64><<<grid, 128, 0, st>>>(qkv, ld, Hq, Hkv, max_len, slot, level, T, inv_freq, scale, Kc, Vc, attn, attn_h, lo_rows);
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ log-softmax + top-k
// One CTA per node: maximum, log-sum-exp, then the `topk` largest logits one after the other.  The packed key
// orders by value, then by lower token id, and every round takes the largest key below the previous one, so
// equal logits come out in token order.
__device__ __forceinline__ float block_reduce_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < 8; ++w) r = fmaxf(r, red[w]);
    return r;
}
__device__ __forceinline__ float block_reduce_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = 0.f;
    for (int w = 0; w < 8; ++w) r += red[w];
    return r;
}
#define TREE_PIECE 4096          // logits of a node that one CTA covers (16 per thread, kept in registers)
int tree_topk_pieces(int V) { return (V + TREE_PIECE - 1) / TREE_PIECE; }

// One CTA per (piece of the row, node): the piece's maximum and sum of exp(x - max), and its `topk` largest keys, largest
// first.  A thread keeps its 16 logits in registers and its current best key; a round takes the block's best, and only the
// thread that owned it looks for its next one.
__global__ void __launch_bounds__(256) tree_topk_piece_kernel(const float* logits, int V, int topk, float2* piece_stats,
                                                              u64* piece_keys) {
    __shared__ float red[8];
    __shared__ u64 kred[8];
    const int piece = blockIdx.x, j = blockIdx.y, pieces = gridDim.x;
    const float* x = logits + (long long)j * V;
    const int c0 = piece * TREE_PIECE;
    u64 key[TREE_PIECE / 256];
    float v[TREE_PIECE / 256];
    float mx = -INFINITY;
#pragma unroll
    for (int t = 0; t < TREE_PIECE / 256; ++t) {
        const int i = c0 + t * 256 + threadIdx.x;
        v[t] = i < V ? x[i] : -INFINITY;
        key[t] = i < V ? pack_key(v[t], i) : 0ull;
        mx = fmaxf(mx, v[t]);
    }
    mx = block_reduce_max(mx, red);
    float se = 0.f;
#pragma unroll
    for (int t = 0; t < TREE_PIECE / 256; ++t) se += expf(v[t] - mx);          // exp(-inf) = 0 beyond the row
    se = block_reduce_sum(se, red);
    if (threadIdx.x == 0) piece_stats[(long long)j * pieces + piece] = make_float2(mx, se);
    u64 mine = 0;
#pragma unroll
    for (int t = 0; t < TREE_PIECE / 256; ++t) mine = key[t] > mine ? key[t] : mine;
    u64* out = piece_keys + ((long long)j * pieces + piece) * TREE_MAX_TOPK;
    for (int r = 0; r < topk; ++r) {
        u64 best = mine;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        __syncthreads();
        if ((threadIdx.x & 31) == 0) kred[threadIdx.x >> 5] = best;
        __syncthreads();
        best = kred[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) best = kred[w] > best ? kred[w] : best;
        if (threadIdx.x == 0) out[r] = best;
        if (best != 0ull && mine == best) {         // keys are unique (they carry the token id): one owner
            mine = 0;
#pragma unroll
            for (int t = 0; t < TREE_PIECE / 256; ++t) {
                if (key[t] == best) key[t] = 0ull;
                mine = key[t] > mine ? key[t] : mine;
            }
        }
    }
}

// One warp per node: log-sum-exp of the row from its pieces, then the `topk` largest of the pieces' keys.  The packed key
// orders by value, then by lower token id, so equal logits come out in token order.
__global__ void __launch_bounds__(32) tree_topk_merge_kernel(const float* logits, int V, int topk, int pieces,
                                                             const float2* piece_stats, const u64* piece_keys, TreeBufs T) {
    const int j = blockIdx.x, lane = threadIdx.x;
    const float* x = logits + (long long)j * V;
    const float2* ps = piece_stats + (long long)j * pieces;
    float mx = -INFINITY;
    for (int c = lane; c < pieces; c += 32) mx = fmaxf(mx, ps[c].x);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float se = 0.f;
    for (int c = lane; c < pieces; c += 32) se += ps[c].y * expf(ps[c].x - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    const float lse = mx + logf(se);
    // every piece's list is sorted: a lane walks the lists of its pieces from their heads
    const u64* pk = piece_keys + (long long)j * pieces * TREE_MAX_TOPK;
    u64 prev = ~0ull;
    for (int r = 0; r < topk; ++r) {
        u64 best = 0;
        for (int c = lane; c < pieces; c += 32)
            for (int t = 0; t < topk; ++t) {
                const u64 key = pk[c * TREE_MAX_TOPK + t];
                if (key < prev) {                     // the first not yet taken of this piece
                    best = key > best ? key : best;
                    break;
                }
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        prev = best;
        if (lane == 0) {
            const int tok = best ? key_index(best) : 0;
            T.top_tok[j * TREE_MAX_TOPK + r] = tok;
            T.top_lp[j * TREE_MAX_TOPK + r] = x[tok] - lse;
        }
    }
}
cudaError_t launch_tree_topk(int nb, const float* logits, int V, int topk, const TreeBufs& T, cudaStream_t st) {
    const int pieces = tree_topk_pieces(V);
    tree_topk_piece_kernel<<<dim3((unsigned)pieces, (unsigned)nb), 256, 0, st>>>(logits, V, topk, T.piece_stats, T.piece_keys);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    tree_topk_merge_kernel<<<nb, 32, 0, st>>>(logits, V, topk, pieces, T.piece_stats, T.piece_keys, T);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ next frontier
// The nb * topk children of this level become candidates (creation order: frontier order, then rank); unless this was
// the last level, the `topk` of them with the highest cumulative log-probability (earlier candidate first among
// equals) form the next frontier, kept in creation order.
__global__ void __launch_bounds__(256) tree_select_kernel(int level, int depth, int nb, int topk, TreeBufs T) {
    __shared__ float s_score[256];
    __shared__ int s_sel[256];
    __shared__ int s_anc[TREE_MAX_TOPK][TREE_MAX_DEPTH], s_store[TREE_MAX_TOPK], s_cand[TREE_MAX_TOPK];
    const int i = threadIdx.x, n = nb * topk;
    const int base = *T.cand_n;
    const int j = i / topk, r = i % topk;
    if (i < TREE_MAX_TOPK * TREE_MAX_DEPTH) s_anc[i / TREE_MAX_DEPTH][i % TREE_MAX_DEPTH] = T.fr_anc[i];
    if (i < TREE_MAX_TOPK) { s_store[i] = T.fr_store[i]; s_cand[i] = T.fr_cand[i]; }
    float score = -INFINITY;
    int tok = 0;
    if (i < n) {
        tok = T.top_tok[j * TREE_MAX_TOPK + r];
        score = T.fr_score[j] + T.top_lp[j * TREE_MAX_TOPK + r];
        T.cand_tok[base + i] = tok;
        T.cand_par[base + i] = T.fr_cand[j];
        T.cand_depth[base + i] = level + 1;
        T.cand_score[base + i] = score;
        T.cand_store[base + i] = -1;
    }
    s_score[i] = score;
    __syncthreads();
    int sel = 0;
    if (i < n && level + 1 < depth) {
        int rank = 0;
        for (int o = 0; o < n; ++o) rank += (s_score[o] > score || (s_score[o] == score && o < i)) ? 1 : 0;
        sel = rank < topk ? 1 : 0;
    }
    s_sel[i] = sel;
    __syncthreads();
    if (sel) {
        int pos = 0;
        for (int o = 0; o < i; ++o) pos += s_sel[o];
        const int store = 1 + level * topk + pos;              // the node joins the frontier of level + 1
        T.fr_cand[pos] = base + i;
        T.fr_tok[pos] = tok;
        T.fr_score[pos] = score;
        T.fr_pslot[pos] = j;
        T.fr_store[pos] = store;
        for (int a = 0; a < level; ++a) T.fr_anc[pos * TREE_MAX_DEPTH + a] = s_anc[j][a];
        T.fr_anc[pos * TREE_MAX_DEPTH + level] = s_store[j];   // the parent's row (the root's when level == 0)
        T.cand_store[base + i] = store;
    }
    if (i == 0) *T.cand_n = base + n;
}
cudaError_t launch_tree_select(int level, int depth, int nb, int topk, const TreeBufs& T, cudaStream_t st) {
    tree_select_kernel<<<1, 256, 0, st>>>(level, depth, nb, topk, T);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ final ranking
// Of all candidates the `keep` with the highest score (earlier candidate first among equals) are the draft tree,
// listed in creation order, parents re-numbered within the list.
__global__ void __launch_bounds__(1024) tree_finalize_kernel(int keep, TreeBufs T, int32_t* out_tokens, int32_t* out_parents,
                                                             float* out_scores, int32_t* out_count) {
    const int n = *T.cand_n;
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const float sc = T.cand_score[i];
        int rank = 0;
        for (int o = 0; o < n; ++o) {
            const float so = T.cand_score[o];
            rank += (so > sc || (so == sc && o < i)) ? 1 : 0;
        }
        T.cand_keep[i] = rank < keep ? 1 : 0;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        int pos = 0;
        for (int o = 0; o < i; ++o) pos += T.cand_keep[o];
        T.cand_pos[i] = T.cand_keep[i] ? pos : -1;
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int pos = T.cand_pos[i];
        if (pos < 0) continue;
        const int par = T.cand_par[i];
        const int pp = par < 0 ? -1 : T.cand_pos[par];
        T.kept_tok[pos] = T.cand_tok[i];
        T.kept_par[pos] = pp;
        T.kept_store[pos] = T.cand_store[i];
        out_tokens[pos] = T.cand_tok[i];
        out_parents[pos] = pp;
        out_scores[pos] = T.cand_score[i];
    }
    if (threadIdx.x == 0) {
        const int cnt = n < keep ? n : keep;
        *T.kept_n = cnt;
        if (out_count) *out_count = cnt;
    }
}
cudaError_t launch_tree_finalize(int keep, const TreeBufs& T, int32_t* out_tokens, int32_t* out_parents, float* out_scores,
                                 int32_t* out_count, cudaStream_t st) {
    tree_finalize_kernel<<<1, 1024, 0, st>>>(keep, T, out_tokens, out_parents, out_scores, out_count);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ verification
template <typename LT>
__global__ void __launch_bounds__(256) tree_row_argmax_kernel(const void* logits, int V, u64* keys) {
    __shared__ u64 kred[8];
    const LT* row = (const LT*)logits + (long long)blockIdx.y * V;
    const int c0 = blockIdx.x * 2048, c1 = min(V, c0 + 2048);
    u64 best = 0;
    for (int i = c0 + threadIdx.x; i < c1; i += 256) {
        const u64 kk = pack_key(load_as_float<LT>(row, i), i);
        best = kk > best ? kk : best;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((threadIdx.x & 31) == 0) kred[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 m = kred[0];
        for (int w = 1; w < 8; ++w) m = kred[w] > m ? kred[w] : m;
        atomicMax(keys + blockIdx.y, m);
    }
}

// The walk: from the root, follow the child that carries the target's argmax for as long as there is one.  Then
// the K/V rows of the accepted nodes that have one are moved right behind the root's row, in path order (a row's
// destination never lies beyond its source, and the moves are made one after the other), and the slot gets its new
// row count.
template <typename WT>
__global__ void __launch_bounds__(256) tree_walk_kernel(int slot, int depth, int Hkv, int dh, int max_len, TreeBufs T,
                                                        const u64* keys, void* Kc, void* Vc, int* kv_len, int32_t* out_accept,
                                                        int32_t* out_path, int32_t* out_next, int32_t* out_kv_len) {
    __shared__ int s_path[TREE_MAX_DEPTH], s_n, s_rows;
    const int n = *T.kept_n, P = *T.P;
    if (threadIdx.x == 0) {
        int cur = -1, acc = 0, t = 0;
        for (;;) {
            t = key_index(keys[cur + 1]);
            int nxt = -1;
            for (int i = 0; i < n; ++i)
                if (T.kept_par[i] == cur && T.kept_tok[i] == t) { nxt = i; break; }
            if (nxt < 0 || acc >= depth) break;
            cur = nxt;
            s_path[acc++] = cur;
        }
        int rows = 0;
        while (rows < acc && T.kept_store[s_path[rows]] >= 0) ++rows;
        s_n = acc;
        s_rows = rows;
        *out_accept = acc;
        *out_next = t;
        for (int i = 0; i < depth; ++i) out_path[i] = i < acc ? s_path[i] : -1;
        kv_len[slot] = P + 1 + rows;
        if (out_kv_len) *out_kv_len = P + 1 + rows;
    }
    __syncthreads();
    const int rows = s_rows, kvw = Hkv * dh;
    for (int m = 0; m < rows; ++m) {
        const int src = P + T.kept_store[s_path[m]], dst = P + 1 + m;
        if (src == dst) continue;                               // uniform over the CTA
        for (int i0 = 0; i0 < kvw; i0 += 256) {
            const int i = i0 + threadIdx.x;
            float kx = 0.f, vx = 0.f;
            long long od = 0;
            if (i < kvw) {
                const int h = i / dh, e = i % dh;
                const long long os = (((long long)slot * Hkv + h) * max_len + src) * dh + e;
                od = (((long long)slot * Hkv + h) * max_len + dst) * dh + e;
                kx = load_as_float<WT>(Kc, os);
                vx = load_as_float<WT>(Vc, os);
            }
            if (i < kvw) {
                store_from_float<WT>(Kc, od, kx);
                store_from_float<WT>(Vc, od, vx);
            }
        }
        __syncthreads();
    }
}

cudaError_t launch_tree_verify(int dtype, int logits_dtype, int slot, int depth, int rows, int V, int Hkv, int dh, int max_len,
                               const TreeBufs& T, const void* logits, void* Kc, void* Vc, int* kv_len, int32_t* out_accept,
                               int32_t* out_path, int32_t* out_next, int32_t* out_kv_len, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(T.row_keys, 0, sizeof(u64) * rows, st);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((V + 2047) / 2048), (unsigned)rows);
    if (logits_dtype == HIVIS_BF16) tree_row_argmax_kernel<bf16><<<grid, 256, 0, st>>>(logits, V, T.row_keys);
    else tree_row_argmax_kernel<float><<<grid, 256, 0, st>>>(logits, V, T.row_keys);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (dtype == HIVIS_BF16)
        tree_walk_kernel<bf16><<<1, 256, 0, st>>>(slot, depth, Hkv, dh, max_len, T, T.row_keys, Kc, Vc, kv_len, out_accept, out_path, out_next, out_kv_len);
    else
        tree_walk_kernel<float><<<1, 256, 0, st>>>(slot, depth, Hkv, dh, max_len, T, T.row_keys, Kc, Vc, kv_len, out_accept, out_path, out_next, out_kv_len);
    return cudaGetLastError();
}
