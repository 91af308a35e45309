// Verification of a chained draft by speculative sampling (temperature > 0): the drafted token of step j is kept
// with probability min(1, p_j(x) / q_j(x)), p and q the target's and the drafter's softmax at that step; the first
// token that is not kept and all after it are dropped and the next token is drawn from the normalised max(0, p - q)
// (from p of the last row when every token was kept).  The uniform numbers come from the caller.
#include "attn_body.cuh"

#define SV_SPAN 4096            // logits of a row that one CTA of the statistics kernel covers (16 per thread, kept in registers)
#define SV_THREADS 1024         // threads per sequence in the decision kernel
#define SV_CHUNK 1024           // tokens per chunk of the inverse CDF (one warp sums a chunk)
#define SV_MAX_CHUNKS 1024

// Pieces of a row: piece c covers logits [c * SV_SPAN, min(V, (c + 1) * SV_SPAN)).
__host__ __device__ __forceinline__ int sv_pieces(int V) { return (V + SV_SPAN - 1) / SV_SPAN; }

// One CTA per piece of a logits row: its maximum and the sum of exp((x - max) / T), each logit read once.
// Rows [0, n_target) are the target's (type LT), rows [n_target, n_target + n_draft) the drafter's (fp32).
template <typename LT>
__global__ void __launch_bounds__(256) row_stats_kernel(const void* target, const float* draft, int n_target, int V,
                                                        float inv_t, float2* part) {
    __shared__ float redf[8];
    const int r = blockIdx.y, c0 = blockIdx.x * SV_SPAN;
    const bool is_t = r < n_target;
    const LT* tr = (const LT*)target + (long long)r * V;
    const float* dr = draft + (long long)(r - n_target) * V;
    float x[SV_SPAN / 256];
    float mx = -INFINITY;
    // 16-byte loads where the rows start on 16-byte boundaries (V a multiple of 8; a vector is then inside the row or beyond it)
    const bool vec = (V & 7) == 0;
    if (vec && is_t && sizeof(LT) == 2) {
        const uint4* src = (const uint4*)((const bf16*)target + (long long)r * V + c0);
#pragma unroll
        for (int j = 0; j < SV_SPAN / 2048; ++j) {
            const int vi = j * 256 + threadIdx.x;
            if (c0 + vi * 8 < V) {
                const uint4 w = __ldg(src + vi);
                x[8 * j + 0] = bf16_lo(w.x); x[8 * j + 1] = bf16_hi(w.x); x[8 * j + 2] = bf16_lo(w.y); x[8 * j + 3] = bf16_hi(w.y);
                x[8 * j + 4] = bf16_lo(w.z); x[8 * j + 5] = bf16_hi(w.z); x[8 * j + 6] = bf16_lo(w.w); x[8 * j + 7] = bf16_hi(w.w);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[8 * j + e] = -INFINITY;
            }
        }
    } else if (vec && (!is_t || sizeof(LT) == 4)) {
        const float4* src = (const float4*)((is_t ? (const float*)target + (long long)r * V : dr) + c0);
#pragma unroll
        for (int j = 0; j < SV_SPAN / 1024; ++j) {
            const int vi = j * 256 + threadIdx.x;
            if (c0 + vi * 4 < V) {
                const float4 w = __ldg(src + vi);
                x[4 * j + 0] = w.x; x[4 * j + 1] = w.y; x[4 * j + 2] = w.z; x[4 * j + 3] = w.w;
            } else {
                x[4 * j + 0] = x[4 * j + 1] = x[4 * j + 2] = x[4 * j + 3] = -INFINITY;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < SV_SPAN / 256; ++j) {
            const int i = c0 + j * 256 + threadIdx.x;
            x[j] = i < V ? (is_t ? load_as_float<LT>(tr, i) : __ldg(dr + i)) : -INFINITY;
        }
    }
#pragma unroll
    for (int j = 0; j < SV_SPAN / 256; ++j) mx = fmaxf(mx, x[j]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((threadIdx.x & 31) == 0) redf[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = redf[0];
#pragma unroll
    for (int w = 1; w < 8; ++w) mx = fmaxf(mx, redf[w]);
    __syncthreads();
    float se = 0.f;
#pragma unroll
    for (int j = 0; j < SV_SPAN / 256; ++j) se += expf((x[j] - mx) * inv_t);         // exp(-inf) = 0 beyond the row
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) se += __shfl_xor_sync(0xffffffffu, se, o);
    if ((threadIdx.x & 31) == 0) redf[threadIdx.x >> 5] = se;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
#pragma unroll
        for (int w = 0; w < 8; ++w) t += (double)redf[w];
        part[(long long)r * gridDim.x + blockIdx.x] = make_float2(mx, (float)t);
    }
}

// (max, log sum exp((x - max) / T)) of a row from its pieces
__device__ __forceinline__ float2 sv_row_stats(const float2* part, int pieces, float inv_t) {
    float mx = -INFINITY;
    for (int c = 0; c < pieces; ++c) mx = fmaxf(mx, part[c].x);
    double se = 0.0;
    for (int c = 0; c < pieces; ++c) se += (double)part[c].y * (double)expf((part[c].x - mx) * inv_t);
    return make_float2(mx, (float)log(se));
}

// One CTA per sequence: acceptance tests, then the draw of the next token by inverse CDF, then the rollback.
// The masses of the row that is drawn from are summed per chunk of 1024 tokens (a warp per chunk, fixed order), the
// chunk that holds u * total is found from the chunk sums and only that chunk is scanned.
template <typename LT>
__global__ void __launch_bounds__(SV_THREADS) sampled_verify_kernel(SlotList sl, int k, int V, float inv_t,
                                                                    const int32_t* draft_ids, const float* draft,
                                                                    const void* target, const float2* part,
                                                                    const float* u_accept, const float* u_sample, int* kv_len,
                                                                    int32_t* out_accept, int32_t* out_next,
                                                                    int32_t* out_kv_len) {
    __shared__ float2 s_st[2 * HIVIS_MAX_K + 1];      // rows 0..k: the target's, k+1..2k: the drafter's
    __shared__ int s_acc[HIVIS_MAX_K], s_n, s_found, s_chunk, s_clast, s_last[SV_THREADS / 32];
    __shared__ double s_sum[SV_MAX_CHUNKS], s_base, s_tot;
    __shared__ float s_warp[SV_THREADS / 32];
    const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, B = sl.n;
    const int pieces = sv_pieces(V);
    if (tid < 2 * k + 1) {
        const long long row = tid <= k ? (long long)b * (k + 1) + tid : (long long)B * (k + 1) + (long long)b * k + (tid - k - 1);
        s_st[tid] = sv_row_stats(part + row * pieces, pieces, inv_t);
    }
    __syncthreads();
    if (tid < k) {
        const int x = draft_ids[(long long)b * k + tid];
        const LT* tr = (const LT*)target + ((long long)b * (k + 1) + tid) * V;
        const float* dr = draft + ((long long)b * k + tid) * V;
        int ok = 0;
        if (x >= 0 && x < V) {
            const float lp = (load_as_float<LT>(tr, x) - s_st[tid].x) * inv_t - s_st[tid].y;
            const float lq = (dr[x] - s_st[k + 1 + tid].x) * inv_t - s_st[k + 1 + tid].y;
            const float a = expf(fminf(0.f, lp - lq));
            ok = u_accept[(long long)b * k + tid] < a ? 1 : 0;
        }
        s_acc[tid] = ok;
    }
    __syncthreads();
    if (tid == 0) {
        int n = 0;
        while (n < k && s_acc[n]) ++n;
        s_n = n;
        s_found = V;
        s_clast = -1;
    }
    __syncthreads();
    const int n = s_n;
    const LT* tr = (const LT*)target + ((long long)b * (k + 1) + n) * V;
    const float* dr = draft + ((long long)b * k + (n < k ? n : 0)) * V;
    const float mt = s_st[n].x, lt = s_st[n].y;
    const float md = n < k ? s_st[k + 1 + n].x : 0.f, ld = n < k ? s_st[k + 1 + n].y : 0.f;
    auto mass = [&](int i, bool resid) {
        const float p = expf((load_as_float<LT>(tr, i) - mt) * inv_t - lt);
        if (!resid) return p;
        const float q = expf((__ldg(dr + i) - md) * inv_t - ld);
        return fmaxf(p - q, 0.f);
    };
    // four consecutive tokens at once (rows on 16-byte boundaries when V is a multiple of 8)
    const bool vec = (V & 7) == 0;
    auto mass4 = [&](int i, bool resid, float (&m)[4]) {
        float lt4[4], ld4[4];
        if (vec && i + 3 < V) {
            if constexpr (sizeof(LT) == 2) {
                const uint2 w = __ldg((const uint2*)((const bf16*)tr + i));
                lt4[0] = bf16_lo(w.x); lt4[1] = bf16_hi(w.x); lt4[2] = bf16_lo(w.y); lt4[3] = bf16_hi(w.y);
            } else {
                const float4 w = __ldg((const float4*)((const float*)tr + i));
                lt4[0] = w.x; lt4[1] = w.y; lt4[2] = w.z; lt4[3] = w.w;
            }
            if (resid) {
                const float4 w = __ldg((const float4*)(dr + i));
                ld4[0] = w.x; ld4[1] = w.y; ld4[2] = w.z; ld4[3] = w.w;
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float p = expf((lt4[e] - mt) * inv_t - lt);
                m[e] = resid ? fmaxf(p - expf((ld4[e] - md) * inv_t - ld), 0.f) : p;
            }
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) m[e] = i + e < V ? mass(i + e, resid) : 0.f;
        }
    };
    const int nchunks = (V + SV_CHUNK - 1) / SV_CHUNK;
    bool resid = n < k;
    int last_pos = -1;
    for (int pass = 0; pass < 2; ++pass) {
        // chunk sums: lane l of the chunk's warp takes tokens 4 l .. 4 l + 3 of every 128
        last_pos = -1;
        for (int c = warp; c < nchunks; c += SV_THREADS / 32) {
            double acc = 0.0;
#pragma unroll
            for (int j = 0; j < SV_CHUNK / 128; ++j) {
                float loc = 0.f, m4[4];
                const int i0 = c * SV_CHUNK + j * 128 + lane * 4;
                mass4(i0, resid, m4);
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (m4[e] > 0.f) last_pos = i0 + e;
                    loc += m4[e];
                }
                acc += (double)loc;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) s_sum[c] = acc;
        }
        __syncthreads();
        if (tid == 0) {
            double tot = 0.0;
            for (int c = 0; c < nchunks; ++c) tot += s_sum[c];
            s_tot = tot;
        }
        __syncthreads();
        // p == q exactly: nothing is left over (and such a token is never rejected): draw from p
        if (!(resid && !(s_tot > 0.0))) break;
        __syncthreads();
        resid = false;
    }
    const double want = (double)u_sample[b] * s_tot;
    if (tid == 0) {
        double run = 0.0;
        int c = 0;
        for (; c < nchunks - 1; ++c) {
            if (run + s_sum[c] > want) break;
            run += s_sum[c];
        }
        s_chunk = c;
        s_base = run;
    }
    __syncthreads();
    {
        // the chunk that holds the wanted mass: four consecutive tokens per thread, an exclusive scan over the block
        const int c0 = s_chunk * SV_CHUNK;
        float m[4] = {0.f, 0.f, 0.f, 0.f}, loc = 0.f;
        if (tid < SV_CHUNK / 4) mass4(c0 + tid * 4, resid, m);
#pragma unroll
        for (int e = 0; e < 4; ++e) loc += m[e];
        // (should rounding keep the scan below the wanted mass although the chunk sums said it is here: the chunk's
        // last token with mass)
        if (loc > 0.f) atomicMax(&s_clast, c0 + tid * 4 + (m[3] > 0.f ? 3 : m[2] > 0.f ? 2 : m[1] > 0.f ? 1 : 0));
        float incl = loc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
        }
        if (lane == 31) s_warp[warp] = incl;
        __syncthreads();
        float wbase = 0.f;
        for (int w = 0; w < warp; ++w) wbase += s_warp[w];
        double run = s_base + (double)wbase + (double)(incl - loc);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            run += (double)m[e];
            if (run > want && m[e] > 0.f) {
                atomicMin(&s_found, c0 + tid * 4 + e);
                break;
            }
        }
    }
    // rounding may leave the cumulative sum a hair below u * total: the last token with mass
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
    if (lane == 0) s_last[warp] = last_pos;
    __syncthreads();
    if (tid == 0) {
        int lp = s_last[0];
        for (int w = 1; w < SV_THREADS / 32; ++w) lp = max(lp, s_last[w]);
        const int next = s_found < V ? s_found : (s_chunk < nchunks - 1 && s_clast >= 0) ? s_clast : (lp >= 0 ? lp : 0);
        const int slot = sl.slot[b];
        const int pairs = kv_len[slot] - k + 1;
        const int rows = pairs + (n < k - 1 ? n : k - 1);
        kv_len[slot] = rows;
        out_accept[b] = n;
        out_next[b] = next;
        if (out_kv_len) out_kv_len[b] = rows;
    }
}

cudaError_t launch_verify_sampled(int logits_dtype, const SlotList& sl, int k, int V, float temperature,
                                  const int32_t* draft_ids, const float* draft_logits, const void* target_logits,
                                  float2* stats, const float* u_accept, const float* u_sample, int* kv_len,
                                  int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len, cudaStream_t st) {
    const int B = sl.n, nt = B * (k + 1), nd = B * k;
    const float inv_t = 1.0f / temperature;
    if ((V + SV_CHUNK - 1) / SV_CHUNK > SV_MAX_CHUNKS) return cudaErrorInvalidValue;
    const dim3 grid((unsigned)sv_pieces(V), (unsigned)(nt + nd));
    if (logits_dtype == HIVIS_BF16) row_stats_kernel<bf16><<<grid, 256, 0, st>>>(target_logits, draft_logits, nt, V, inv_t, stats);
    else row_stats_kernel<float><<<grid, 256, 0, st>>>(target_logits, draft_logits, nt, V, inv_t, stats);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (logits_dtype == HIVIS_BF16)
        sampled_verify_kernel<bf16><<<B, SV_THREADS, 0, st>>>(sl, k, V, inv_t, draft_ids, draft_logits, target_logits, stats,
                                                               u_accept, u_sample, kv_len, out_accept, out_next, out_kv_len);
    else
        sampled_verify_kernel<float><<<B, SV_THREADS, 0, st>>>(sl, k, V, inv_t, draft_ids, draft_logits, target_logits, stats,
                                                                u_accept, u_sample, kv_len, out_accept, out_next, out_kv_len);
    return cudaGetLastError();
}

int sampled_stats_entries(int max_batch, int max_k, int V) { return max_batch * (2 * max_k + 1) * sv_pieces(V); }
