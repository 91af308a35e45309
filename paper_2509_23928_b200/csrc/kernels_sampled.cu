// Verification of a chained draft by speculative sampling (temperature > 0): the drafted token of step j is kept
// with probability min(1, p_j(x) / q_j(x)), p and q the target's and the drafter's softmax at that step; the first
// token that is not kept and all after it are dropped and the next token is drawn from the normalised max(0, p - q)
// (from p of the last row when every token was kept).  The uniform numbers come from the caller.
#include "attn_body.cuh"

__device__ __forceinline__ float sblock_max(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float r = red[0];
    for (int w = 1; w < 8; ++w) r = fmaxf(r, red[w]);
    return r;
}
__device__ __forceinline__ double sblock_sum(double v, double* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    double r = 0.0;
    for (int w = 0; w < 8; ++w) r += red[w];
    return r;
}

// One CTA per logits row: its maximum and the logarithm of the sum of exp((x - max) / T).
// Rows [0, n_target) are the target's (type LT), rows [n_target, n_target + n_draft) the drafter's (fp32).
template <typename LT>
__global__ void __launch_bounds__(256) row_stats_kernel(const void* target, const float* draft, int n_target, int V,
                                                        float inv_t, float2* stats) {
    __shared__ float redf[8];
    __shared__ double redd[8];
    const int r = blockIdx.x;
    const bool is_t = r < n_target;
    const LT* tr = (const LT*)target + (long long)r * V;
    const float* dr = draft + (long long)(r - n_target) * V;
    float mx = -INFINITY;
    for (int i = threadIdx.x; i < V; i += 256) mx = fmaxf(mx, is_t ? load_as_float<LT>(tr, i) : dr[i]);
    mx = sblock_max(mx, redf);
    double se = 0.0;
    for (int i = threadIdx.x; i < V; i += 256) se += (double)expf(((is_t ? load_as_float<LT>(tr, i) : dr[i]) - mx) * inv_t);
    se = sblock_sum(se, redd);
    if (threadIdx.x == 0) stats[r] = make_float2(mx, (float)log(se));
}

// One CTA per sequence: acceptance tests, then the draw of the next token by inverse CDF, then the rollback.
template <typename LT>
__global__ void __launch_bounds__(256) sampled_verify_kernel(SlotList sl, int k, int V, float inv_t, const int32_t* draft_ids,
                                                             const float* draft, const void* target, const float2* stats,
                                                             const float* u_accept, const float* u_sample, int* kv_len,
                                                             int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len) {
    __shared__ int s_acc[HIVIS_MAX_K], s_n, s_found;
    __shared__ double redd[8];
    __shared__ float s_warp[8];
    __shared__ double s_base;
    const int b = blockIdx.x, tid = threadIdx.x, B = sl.n;
    const float2* st_t = stats + (long long)b * (k + 1);
    const float2* st_d = stats + (long long)B * (k + 1) + (long long)b * k;
    if (tid < k) {
        const int x = draft_ids[(long long)b * k + tid];
        const LT* tr = (const LT*)target + ((long long)b * (k + 1) + tid) * V;
        const float* dr = draft + ((long long)b * k + tid) * V;
        int ok = 0;
        if (x >= 0 && x < V) {
            const float lp = (load_as_float<LT>(tr, x) - st_t[tid].x) * inv_t - st_t[tid].y;
            const float lq = (dr[x] - st_d[tid].x) * inv_t - st_d[tid].y;
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
        s_base = 0.0;
    }
    __syncthreads();
    const int n = s_n;
    const LT* tr = (const LT*)target + ((long long)b * (k + 1) + n) * V;
    const float* dr = draft + ((long long)b * k + (n < k ? n : 0)) * V;
    const float mt = st_t[n].x, lt = st_t[n].y;
    const float md = n < k ? st_d[n].x : 0.f, ld = n < k ? st_d[n].y : 0.f;
    auto pmass = [&](int i) { return expf((load_as_float<LT>(tr, i) - mt) * inv_t - lt); };
    auto mass = [&](int i, bool resid) {
        const float p = pmass(i);
        if (!resid) return p;
        const float q = expf((dr[i] - md) * inv_t - ld);
        return fmaxf(p - q, 0.f);
    };
    bool resid = n < k;
    double tot = 0.0;
    for (int i = tid; i < V; i += 256) tot += (double)mass(i, resid);
    tot = sblock_sum(tot, redd);
    if (resid && !(tot > 0.0)) {            // p == q exactly: nothing is left over (and such a token is never rejected)
        resid = false;
        tot = 0.0;
        for (int i = tid; i < V; i += 256) tot += (double)pmass(i);
        tot = sblock_sum(tot, redd);
    }
    const double want = (double)u_sample[b] * tot;
    // inverse CDF: chunks of 256 x 4 consecutive tokens, an exclusive scan inside the chunk, a running base across chunks
    int last_pos = -1;
    for (int c0 = 0; c0 < V && s_found == V; c0 += 1024) {
        float m[4];
        float loc = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = c0 + tid * 4 + e;
            m[e] = i < V ? mass(i, resid) : 0.f;
            if (m[e] > 0.f) last_pos = i;
            loc += m[e];
        }
        float incl = loc;                   // inclusive scan over the warp
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const float t = __shfl_up_sync(0xffffffffu, incl, o);
            if ((tid & 31) >= o) incl += t;
        }
        if ((tid & 31) == 31) s_warp[tid >> 5] = incl;
        __syncthreads();
        float wbase = 0.f;
        for (int w = 0; w < (tid >> 5); ++w) wbase += s_warp[w];
        double run = s_base + (double)wbase + (double)(incl - loc);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            run += (double)m[e];
            if (run > want && m[e] > 0.f) {
                atomicMin(&s_found, c0 + tid * 4 + e);
                break;
            }
        }
        __syncthreads();
        if (tid == 255) s_base += (double)wbase + (double)incl;
        __syncthreads();
    }
    // rounding may leave the cumulative sum a hair below u * total: the last token with mass
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last_pos = max(last_pos, __shfl_xor_sync(0xffffffffu, last_pos, o));
    __shared__ int s_last[8];
    if ((tid & 31) == 0) s_last[tid >> 5] = last_pos;
    __syncthreads();
    if (tid == 0) {
        int lp = s_last[0];
        for (int w = 1; w < 8; ++w) lp = max(lp, s_last[w]);
        const int next = s_found < V ? s_found : (lp >= 0 ? lp : 0);
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
    if (logits_dtype == HIVIS_BF16) row_stats_kernel<bf16><<<nt + nd, 256, 0, st>>>(target_logits, draft_logits, nt, V, inv_t, stats);
    else row_stats_kernel<float><<<nt + nd, 256, 0, st>>>(target_logits, draft_logits, nt, V, inv_t, stats);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (logits_dtype == HIVIS_BF16)
        sampled_verify_kernel<bf16><<<B, 256, 0, st>>>(sl, k, V, inv_t, draft_ids, draft_logits, target_logits, stats, u_accept,
                                                        u_sample, kv_len, out_accept, out_next, out_kv_len);
    else
        sampled_verify_kernel<float><<<B, 256, 0, st>>>(sl, k, V, inv_t, draft_ids, draft_logits, target_logits, stats, u_accept,
                                                         u_sample, kv_len, out_accept, out_next, out_kv_len);
    return cudaGetLastError();
}
