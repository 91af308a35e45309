// Split-KV decode attention over the ragged text-only cache.
//
// One new position per sequence.  A CTA takes (split, group of GQ query heads sharing one KV head,
// sequence); its four warps walk the split's cache rows 32 at a time:
//   scores : one lane per cache row, the row's K read with 128-bit loads, q broadcast from shared
//            memory (already rotated);
//   softmax: online (running max / sum) with warp shuffles;
//   PV     : one lane per slice of the head dimension, the row's probability broadcast by shuffle.
// The new position's K (rotated here) and V are taken from the QKV output and appended to the cache
// by the CTA whose split contains it.  Each CTA writes an unnormalised partial (max, sum, acc); the
// last CTA to arrive for a (sequence, head group) - found with an arrival counter, nobody waits -
// merges the partials in split order, so the result does not depend on arrival order.
#include "hivis_internal.cuh"

template <typename WT, int DH, int GQ>
__global__ void __launch_bounds__(128) attn_decode_kernel(const AttnArgs a) {
    constexpr int EPL = DH / 32;                     // head-dim elements per lane in the PV phase
    __shared__ float q_s[GQ][DH];
    __shared__ float knew[DH], vnew[DH];
    __shared__ float m_s[4][GQ], l_s[4][GQ];
    __shared__ float acc_s[4][GQ][DH];
    __shared__ int s_last;

    const int split = blockIdx.x, hg = blockIdx.y, b = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = a.Hq / a.Hkv;
    const int h0 = hg * GQ;                          // first query head of this CTA
    const int kvh = h0 / G;
    const int p = a.pos0[b] + a.step;                // row of the new position
    const int len = p + 1;
    const int nsplits = (len + a.chunk - 1) / a.chunk;
    if (split >= nsplits) return;
    const int r0 = split * a.chunk;
    const int r1 = min(len, r0 + a.chunk);
    const bool owns_new = (p >= r0 && p < r1);
    const int slot = a.slots[b];
    const int half = DH / 2;
    const int qw = a.Hq * DH, kvw = a.Hkv * DH;
    const float* qkv = a.qkv + (long long)b * a.ld;

    // rotate q into shared memory
    for (int i = tid; i < GQ * half; i += 128) {
        const int gq = i / half, j = i % half;
        double sn, cs;
        sincos((double)p * a.inv_freq[j], &sn, &cs);
        const float c = (float)cs, s = (float)sn;
        const float x0 = __ldcg(qkv + (h0 + gq) * DH + j), x1 = __ldcg(qkv + (h0 + gq) * DH + j + half);
        q_s[gq][j] = (x0 * c - x1 * s) * a.scale;
        q_s[gq][j + half] = (x1 * c + x0 * s) * a.scale;
    }
    WT* Kbase = (WT*)a.Kc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
    WT* Vbase = (WT*)a.Vc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
    if (owns_new) {
        const bool writer = (h0 % G) == 0;           // one CTA per KV head appends the row
        for (int j = tid; j < half; j += 128) {
            double sn, cs;
            sincos((double)p * a.inv_freq[j], &sn, &cs);
            const float c = (float)cs, s = (float)sn;
            const float x0 = __ldcg(qkv + qw + kvh * DH + j), x1 = __ldcg(qkv + qw + kvh * DH + j + half);
            float k0 = x0 * c - x1 * s, k1 = x1 * c + x0 * s;
            if (writer) {
                store_from_float<WT>(Kbase, (long long)p * DH + j, k0);
                store_from_float<WT>(Kbase, (long long)p * DH + j + half, k1);
            }
            // attend to exactly what the cache holds (storage rounding included)
            if (sizeof(WT) == 2) {
                k0 = __bfloat162float(__float2bfloat16_rn(k0));
                k1 = __bfloat162float(__float2bfloat16_rn(k1));
            }
            knew[j] = k0;
            knew[j + half] = k1;
        }
        for (int j = tid; j < DH; j += 128) {
            float v = __ldcg(qkv + qw + kvw + kvh * DH + j);
            if (writer) store_from_float<WT>(Vbase, (long long)p * DH + j, v);
            if (sizeof(WT) == 2) v = __bfloat162float(__float2bfloat16_rn(v));
            vnew[j] = v;
        }
    }
    __syncthreads();

    float m_run[GQ], l_run[GQ], acc[GQ][EPL];
#pragma unroll
    for (int gq = 0; gq < GQ; ++gq) {
        m_run[gq] = -INFINITY;
        l_run[gq] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[gq][e] = 0.f;
    }

    for (int base = r0 + warp * 32; base < r1; base += 128) {
        const int trow = base + lane;
        const bool ok = trow < r1;
        float s[GQ];
#pragma unroll
        for (int gq = 0; gq < GQ; ++gq) s[gq] = 0.f;
        if (ok) {
            if (trow == p) {
                for (int i = 0; i < DH; ++i) {
                    const float kv = knew[i];
#pragma unroll
                    for (int gq = 0; gq < GQ; ++gq) s[gq] = fmaf(q_s[gq][i], kv, s[gq]);
                }
            } else {
                const WT* krow = Kbase + (long long)trow * DH;
                constexpr int VEC = 16 / (int)sizeof(WT);
#pragma unroll 4
                for (int c = 0; c < DH / VEC; ++c) {
                    const uint4 w = *((const uint4*)krow + c);
                    float kf[VEC];
                    if constexpr (sizeof(WT) == 2) {
                        kf[0] = bf16_lo(w.x); kf[1] = bf16_hi(w.x); kf[2] = bf16_lo(w.y); kf[3] = bf16_hi(w.y);
                        kf[4] = bf16_lo(w.z); kf[5] = bf16_hi(w.z); kf[6] = bf16_lo(w.w); kf[7] = bf16_hi(w.w);
                    } else {
                        kf[0] = __uint_as_float(w.x); kf[1] = __uint_as_float(w.y);
                        kf[2] = __uint_as_float(w.z); kf[3] = __uint_as_float(w.w);
                    }
#pragma unroll
                    for (int i = 0; i < VEC; ++i)
#pragma unroll
                        for (int gq = 0; gq < GQ; ++gq) s[gq] = fmaf(q_s[gq][c * VEC + i], kf[i], s[gq]);
                }
            }
        }
        // online softmax over this block of 32 rows
        float pr[GQ];
#pragma unroll
        for (int gq = 0; gq < GQ; ++gq) {
            float sv = ok ? s[gq] : -INFINITY;
            float mb = sv;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, o));
            const float mn = fmaxf(m_run[gq], mb);   // finite: the block has at least one valid row
            const float corr = expf(m_run[gq] - mn);
            pr[gq] = ok ? expf(sv - mn) : 0.f;
            float ps = pr[gq];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
            l_run[gq] = l_run[gq] * corr + ps;
            m_run[gq] = mn;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[gq][e] *= corr;
        }
        // PV: lane owns head-dim elements [lane*EPL, +EPL)
        const int nrows = min(32, r1 - base);
        for (int j = 0; j < nrows; ++j) {
            const int tj = base + j;
            float v[EPL];
            if (tj == p) {
#pragma unroll
                for (int e = 0; e < EPL; ++e) v[e] = vnew[lane * EPL + e];
            } else {
                const WT* vrow = Vbase + (long long)tj * DH + lane * EPL;
                if constexpr (sizeof(WT) == 2) {
                    if constexpr (EPL == 4) {
                        const uint2 w = *(const uint2*)vrow;
                        v[0] = bf16_lo(w.x); v[1] = bf16_hi(w.x); v[2] = bf16_lo(w.y); v[3] = bf16_hi(w.y);
                    } else {
                        const unsigned w = *(const unsigned*)vrow;
                        v[0] = bf16_lo(w); v[1] = bf16_hi(w);
                    }
                } else {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) v[e] = ((const float*)vrow)[e];
                }
            }
#pragma unroll
            for (int gq = 0; gq < GQ; ++gq) {
                const float pj = __shfl_sync(0xffffffffu, pr[gq], j);
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[gq][e] = fmaf(pj, v[e], acc[gq][e]);
            }
        }
    }
    // merge the four warps
#pragma unroll
    for (int gq = 0; gq < GQ; ++gq) {
        if (lane == 0) {
            m_s[warp][gq] = m_run[gq];
            l_s[warp][gq] = l_run[gq];
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc_s[warp][gq][lane * EPL + e] = acc[gq][e];
    }
    __syncthreads();
    const bool single = nsplits == 1;
    for (int i = tid; i < GQ * DH; i += 128) {
        const int gq = i / DH, dd = i % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, m_s[w][gq]);
        float L = 0.f, A = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float f = m_s[w][gq] == -INFINITY ? 0.f : expf(m_s[w][gq] - M);
            L += l_s[w][gq] * f;
            A += acc_s[w][gq][dd] * f;
        }
        const int h = h0 + gq;
        if (single) {
            const float o = A / L;
            a.attn[(long long)b * qw + h * DH + dd] = o;
            a.attn_h[(long long)b * qw + h * DH + dd] = __float2bfloat16_rn(o);
        } else {
            const long long pi = ((long long)b * a.Hq + h) * a.nsplit + split;
            a.part_acc[pi * DH + dd] = A;
            if (dd == 0) {
                a.part_ml[pi * 2] = M;
                a.part_ml[pi * 2 + 1] = L;
            }
        }
    }
    if (single) return;
    // arrival counter: the last CTA of this (sequence, head group) merges the splits
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        int* ctr = a.counters + (long long)b * a.Hq + h0;
        const int old = atomicAdd(ctr, 1);
        s_last = (old == nsplits - 1);
        if (s_last) *ctr = 0;
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int i = tid; i < GQ * DH; i += 128) {
        const int gq = i / DH, dd = i % DH;
        const int h = h0 + gq;
        const long long p0 = ((long long)b * a.Hq + h) * a.nsplit;
        float M = -INFINITY;
        for (int sp = 0; sp < nsplits; ++sp) M = fmaxf(M, __ldcg(a.part_ml + (p0 + sp) * 2));
        float L = 0.f, A = 0.f;
        for (int sp = 0; sp < nsplits; ++sp) {
            const float f = expf(__ldcg(a.part_ml + (p0 + sp) * 2) - M);
            L += __ldcg(a.part_ml + (p0 + sp) * 2 + 1) * f;
            A += __ldcg(a.part_acc + (p0 + sp) * DH + dd) * f;
        }
        const float o = A / L;
        a.attn[(long long)b * qw + h * DH + dd] = o;
        a.attn_h[(long long)b * qw + h * DH + dd] = __float2bfloat16_rn(o);
    }
}

template <typename WT, int DH>
static cudaError_t launch_attn_g(const AttnArgs& a, cudaStream_t st) {
    const int G = a.Hq / a.Hkv;
    int gq = 1;
    const int cand[5] = {8, 7, 4, 2, 1};
    for (int i = 0; i < 5; ++i)
        if (G % cand[i] == 0) { gq = cand[i]; break; }
    dim3 grid((unsigned)a.nsplit, (unsigned)(a.Hq / gq), (unsigned)a.B);
    switch (gq) {
        case 8: attn_decode_kernel<WT, DH, 8><<<grid, 128, 0, st>>>(a); break;
        case 7: attn_decode_kernel<WT, DH, 7><<<grid, 128, 0, st>>>(a); break;
        case 4: attn_decode_kernel<WT, DH, 4><<<grid, 128, 0, st>>>(a); break;
        case 2: attn_decode_kernel<WT, DH, 2><<<grid, 128, 0, st>>>(a); break;
        default: attn_decode_kernel<WT, DH, 1><<<grid, 128, 0, st>>>(a); break;
    }
    return cudaGetLastError();
}

cudaError_t launch_attention(int dtype, const AttnArgs& a, cudaStream_t st) {
    if (a.B <= 0) return cudaSuccess;
    if (dtype == HIVIS_BF16)
        return a.dh == 128 ? launch_attn_g<bf16, 128>(a, st) : launch_attn_g<bf16, 64>(a, st);
    return a.dh == 128 ? launch_attn_g<float, 128>(a, st) : launch_attn_g<float, 64>(a, st);
}
