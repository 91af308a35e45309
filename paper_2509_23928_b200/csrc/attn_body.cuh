// Body of the split-KV decode attention, shared by the stand-alone kernel (4 warps per unit) and the
// persistent chain kernel (8 warps per unit).  One call handles one unit = (split of the cache rows,
// group of GQ query heads on one KV head, sequence); every thread of the CTA must make the call.
#pragma once
#include "hivis_internal.cuh"

template <int NW, int GQ, int DH>
struct AttnSmem {
    float q_s[GQ][DH];
    float knew[DH], vnew[DH];
    float m_s[NW][GQ], l_s[NW][GQ];
    float acc_s[NW][GQ][DH];
    int s_last;
};

// arrival on a counter: orders this thread's writes, and those of threads it synchronised with before, ahead of
// the addition (release) and the writes of earlier arrivers ahead of what follows (acquire), in one operation
__device__ __forceinline__ int atom_add_acq_rel(int* p, int v) {
    int old;
    asm volatile("atom.acq_rel.gpu.global.add.s32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
    return old;
}
// cos/sin of pos * inv_freq: the product and its reduction to [-pi, pi] are done in double (a few
// instructions), the functions themselves in fp32 on the reduced argument.
__device__ __forceinline__ void rope_cs(int pos, double inv_freq, float& c, float& s) {
    const double ang = (double)pos * inv_freq;
    const double two_pi = 6.283185307179586476925286766559;
    const double r = ang - two_pi * rint(ang * (1.0 / two_pi));
    sincosf((float)r, &s, &c);
}

// Barrier among the NT threads that work on a unit: the whole CTA (BAR == 0) or a named barrier.
template <int BAR, int NT>
__device__ __forceinline__ void attn_sync() {
    if (BAR == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(BAR), "r"(NT) : "memory");
}

// bf16 copy of an attention output element; with lo_rows > 0 the rounding remainder goes to row
// b + lo_rows, so that a bf16 tensor-core operand carries the value to about 16 mantissa bits.
__device__ __forceinline__ void attn_store_h(const AttnArgs& a, int b, int qw, int col, float o) {
    if (!a.attn_h) return;
    const bf16 hi = __float2bfloat16_rn(o);
    a.attn_h[(long long)b * qw + col] = hi;
    if (a.lo_rows > 0) a.attn_h[(long long)(b + a.lo_rows) * qw + col] = __float2bfloat16_rn(o - __bfloat162float(hi));
}

// `tid` is the caller's index among the NW*32 threads that take part (0-based).
template <typename WT, int DH, int GQ, int NW, int BAR = 0>
__device__ __forceinline__ void attn_unit(const AttnArgs& a, int split, int hg, int b, int p, int slot,
                                          AttnSmem<NW, GQ, DH>& sm, int tid = threadIdx.x) {
    constexpr int EPL = DH / 32;                     // head-dim elements per lane in the PV phase
    constexpr int NT = NW * 32;
    constexpr int VEC = 16 / (int)sizeof(WT);
    const int warp = tid >> 5, lane = tid & 31;
    const int G = a.Hq / a.Hkv;
    const int h0 = hg * GQ;                          // first query head of this unit
    const int kvh = h0 / G;
    const int len = p + 1;
    const int nsplits = (len + a.chunk - 1) / a.chunk;
    if (split >= nsplits) return;
    const int r0 = split * a.chunk;
    const int r1 = min(len, r0 + a.chunk);
    const bool owns_new = (p >= r0 && p < r1);
    const int half = DH / 2;
    const int qw = a.Hq * DH, kvw = a.Hkv * DH;
    const float* qkv = a.qkv + (long long)b * a.ld;

    attn_sync<BAR, NT>();                                 // the previous unit's readers are done with sm
    for (int i = tid; i < GQ * half; i += NT) {
        const int gq = i / half, j = i % half;
        float c, s;
        rope_cs(p, a.inv_freq[j], c, s);
        const float x0 = __ldcg(qkv + (h0 + gq) * DH + j), x1 = __ldcg(qkv + (h0 + gq) * DH + j + half);
        sm.q_s[gq][j] = (x0 * c - x1 * s) * a.scale;
        sm.q_s[gq][j + half] = (x1 * c + x0 * s) * a.scale;
    }
    WT* Kbase = (WT*)a.Kc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
    WT* Vbase = (WT*)a.Vc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
    if (owns_new) {
        const bool writer = (h0 % G) == 0;           // one unit per KV head appends the row
        for (int j = tid; j < half; j += NT) {
            float c, s;
            rope_cs(p, a.inv_freq[j], c, s);
            const float x0 = __ldcg(qkv + qw + kvh * DH + j), x1 = __ldcg(qkv + qw + kvh * DH + j + half);
            float k0 = x0 * c - x1 * s, k1 = x1 * c + x0 * s;
            if (writer) {
                store_from_float<WT>(Kbase, (long long)p * DH + j, k0);
                store_from_float<WT>(Kbase, (long long)p * DH + j + half, k1);
            }
            if (sizeof(WT) == 2) {                   // attend to exactly what the cache holds
                k0 = __bfloat162float(__float2bfloat16_rn(k0));
                k1 = __bfloat162float(__float2bfloat16_rn(k1));
            }
            sm.knew[j] = k0;
            sm.knew[j + half] = k1;
        }
        for (int j = tid; j < DH; j += NT) {
            float v = __ldcg(qkv + qw + kvw + kvh * DH + j);
            if (writer) store_from_float<WT>(Vbase, (long long)p * DH + j, v);
            if (sizeof(WT) == 2) v = __bfloat162float(__float2bfloat16_rn(v));
            sm.vnew[j] = v;
        }
    }
    attn_sync<BAR, NT>();

    float m_run[GQ], l_run[GQ], acc[GQ][EPL];
#pragma unroll
    for (int gq = 0; gq < GQ; ++gq) {
        m_run[gq] = -INFINITY;
        l_run[gq] = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[gq][e] = 0.f;
    }

    for (int base = r0 + warp * 32; base < r1; base += NT) {
        const int trow = base + lane;
        const bool ok = trow < r1;
        float s[GQ];
#pragma unroll
        for (int gq = 0; gq < GQ; ++gq) s[gq] = 0.f;
        if (ok) {
            if (trow == p) {
                for (int i = 0; i < DH; ++i) {
                    const float kv = sm.knew[i];
#pragma unroll
                    for (int gq = 0; gq < GQ; ++gq) s[gq] = fmaf(sm.q_s[gq][i], kv, s[gq]);
                }
            } else {
                const uint4* krow = (const uint4*)(Kbase + (long long)trow * DH);
                constexpr int NCH = DH / VEC;
                constexpr int UB = NCH < 16 ? NCH : 16;       // loads in flight per lane
#pragma unroll
                for (int c0 = 0; c0 < NCH; c0 += UB) {
                    uint4 w[UB];
#pragma unroll
                    for (int c = 0; c < UB; ++c) w[c] = krow[c0 + c];
#pragma unroll
                    for (int c = 0; c < UB; ++c) {
                        float kf[VEC];
                        if constexpr (sizeof(WT) == 2) {
                            kf[0] = bf16_lo(w[c].x); kf[1] = bf16_hi(w[c].x); kf[2] = bf16_lo(w[c].y); kf[3] = bf16_hi(w[c].y);
                            kf[4] = bf16_lo(w[c].z); kf[5] = bf16_hi(w[c].z); kf[6] = bf16_lo(w[c].w); kf[7] = bf16_hi(w[c].w);
                        } else {
                            kf[0] = __uint_as_float(w[c].x); kf[1] = __uint_as_float(w[c].y);
                            kf[2] = __uint_as_float(w[c].z); kf[3] = __uint_as_float(w[c].w);
                        }
#pragma unroll
                        for (int i = 0; i < VEC; ++i)
#pragma unroll
                            for (int gq = 0; gq < GQ; ++gq)
                                s[gq] = fmaf(sm.q_s[gq][(c0 + c) * VEC + i], kf[i], s[gq]);
                    }
                }
            }
        }
        // online softmax over this block of 32 rows
        float pr[GQ];
#pragma unroll
        for (int gq = 0; gq < GQ; ++gq) {
            const float sv = ok ? s[gq] : -INFINITY;
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
        // PV: lane owns head-dim elements [lane*EPL, +EPL); V rows are fetched eight at a time
        const int nrows = min(32, r1 - base);
        for (int j0 = 0; j0 < nrows; j0 += 8) {
            float v[8][EPL];
#pragma unroll
            for (int jj = 0; jj < 8; ++jj) {
                const int tj = base + j0 + jj;
                if (j0 + jj >= nrows) {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) v[jj][e] = 0.f;
                } else if (tj == p) {
#pragma unroll
                    for (int e = 0; e < EPL; ++e) v[jj][e] = sm.vnew[lane * EPL + e];
                } else {
                    const WT* vrow = Vbase + (long long)tj * DH + lane * EPL;
                    if constexpr (sizeof(WT) == 2) {
                        if constexpr (EPL == 4) {
                            const uint2 w = *(const uint2*)vrow;
                            v[jj][0] = bf16_lo(w.x); v[jj][1] = bf16_hi(w.x); v[jj][2] = bf16_lo(w.y); v[jj][3] = bf16_hi(w.y);
                        } else {
                            const unsigned w = *(const unsigned*)vrow;
                            v[jj][0] = bf16_lo(w); v[jj][1] = bf16_hi(w);
                        }
                    } else {
#pragma unroll
                        for (int e = 0; e < EPL; ++e) v[jj][e] = ((const float*)vrow)[e];
                    }
                }
            }
#pragma unroll
            for (int jj = 0; jj < 8; ++jj)
#pragma unroll
                for (int gq = 0; gq < GQ; ++gq) {
                    const float pj = __shfl_sync(0xffffffffu, pr[gq], (j0 + jj) & 31);   // 0 beyond nrows
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[gq][e] = fmaf(pj, v[jj][e], acc[gq][e]);
                }
        }
    }
    // merge the warps
#pragma unroll
    for (int gq = 0; gq < GQ; ++gq) {
        if (lane == 0) {
            sm.m_s[warp][gq] = m_run[gq];
            sm.l_s[warp][gq] = l_run[gq];
        }
#pragma unroll
        for (int e = 0; e < EPL; ++e) sm.acc_s[warp][gq][lane * EPL + e] = acc[gq][e];
    }
    attn_sync<BAR, NT>();
    const bool single = nsplits == 1;
    for (int i = tid; i < GQ * DH; i += NT) {
        const int gq = i / DH, dd = i % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) M = fmaxf(M, sm.m_s[w][gq]);
        float L = 0.f, A = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float f = sm.m_s[w][gq] == -INFINITY ? 0.f : expf(sm.m_s[w][gq] - M);
            L += sm.l_s[w][gq] * f;
            A += sm.acc_s[w][gq][dd] * f;
        }
        const int h = h0 + gq;
        if (single) {
            const float o = A / L;
            a.attn[(long long)b * qw + h * DH + dd] = o;
            attn_store_h(a, b, qw, h * DH + dd, o);
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
    // arrival counter: the last unit of this (sequence, head group) merges the splits; nobody waits
    attn_sync<BAR, NT>();
    if (tid == 0) {
        int* ctr = a.counters + (long long)b * a.Hq + h0;
        const int old = atom_add_acq_rel(ctr, 1);
        sm.s_last = (old == nsplits - 1);
        if (sm.s_last) *ctr = 0;
    }
    attn_sync<BAR, NT>();
    if (!sm.s_last) return;
    for (int i = tid; i < GQ * DH; i += NT) {
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
        attn_store_h(a, b, qw, h * DH + dd, o);
    }
}
