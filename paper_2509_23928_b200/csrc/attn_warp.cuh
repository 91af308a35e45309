// Warp-granular split-KV decode attention over the ragged text-only cache (bf16 cache), used by the
// tensor-core chain kernel.
//
// Unit of work: one block of cache rows of one key = (sequence, group of GQ query heads on one KV head).
// The rows a sequence had when the launch began (its prefix, which no draft step changes) are cut into
// blocks of 32; the rows appended by the draft steps of this launch, and the new position itself, form one
// more unit per key, the tail.  The unit list therefore does not depend on the step.  All units of the batch
// are laid out in (sequence, key, block) order and cut into equal contiguous ranges, one per participating
// warp, whatever the sequence lengths: a ragged batch is balanced to within one block.
//
// Prefix blocks are not read from global memory by the warp: a producer thread of the CTA copies each block
// (K rows, then V rows: both are contiguous in the cache) into a stage of the CTA's shared-memory ring with
// bulk copies, far ahead of the warp and independent of any grid barrier, since the prefix is immutable.
// The warp waits for the stage, computes from shared memory and hands the stage back.  The tail unit is
// read with ordinary loads (its rows were written by other CTAs in earlier steps, behind grid barriers); it
// still takes (and returns) an empty ring item so that every unit is exactly one item.
//
// Inside a unit (DH = 128: a cache row is 16 lanes x 16 bytes, so one load instruction reads two whole rows):
//   scores : every lane multiplies its 8-element slice of q with the matching slice of K for the rows it
//            loaded; the slices are summed with a transposing butterfly (15 shuffles for 32 rows), after
//            which each lane holds the complete score of ONE row;
//   softmax: online (running max / sum) with warp shuffles;
//   PV     : lane owns DH/32 output elements; V rows are read as whole rows, the row's probability is
//            broadcast from the lane that holds it.
// A warp keeps accumulating while consecutive units belong to the same key.  When the key changes it writes
// the result - directly if it covered all blocks of the key, else as an unnormalised partial (max, sum, acc)
// to global memory; the warp that completes the key's block count (arrival counter, nobody waits) merges the
// partials in block order, so the result does not depend on arrival order.
// The new position's K (rotated here) and V are appended to the cache by the tail unit.
#pragma once
#include "attn_body.cuh"

struct AttnWArgs {
    const float* qkv;       // [B][ld] fp32: q | k | v of the new position, before RoPE
    int ld;
    bf16* Kc;               // [slot][Hkv][max_len][dh], K stored after RoPE
    bf16* Vc;
    const int* slots;       // [B]
    const int* pos0;        // [B] rows of the sequence when the launch began = cache row of draft step 0
    int step;
    const float2* rope_tab; // [B][dh/2] (cos, sin) of every sequence's new position at this step
    int Hq, Hkv, max_len, B;
    float scale;
    float* part_acc;        // [B][Hq][nslot][dh]
    float* part_ml;         // [B][Hq][nslot][2]
    int nslot;              // >= units of the longest key
    int* counters;          // [B][Hq/GQ] units finished per key, zero between phases
    float* attn;            // [B][Hq*dh] fp32
    bf16* attn_h;           // [B][Hq*dh] bf16 (+ remainder rows when lo_rows > 0)
    int lo_rows;
};

// Unit ranges of the warps.  32-bit arithmetic: units * warps stays far below 2^31 for every size the
// library accepts (<= 16 sequences x 128 head groups x 513 units, a few thousand warps would still fit).
__device__ __forceinline__ unsigned attw_lo(unsigned U, int g, int NW) { return U * (unsigned)g / (unsigned)NW; }
__device__ __forceinline__ int attw_owner(unsigned U, int NW, unsigned u) {
    int g = (int)(u * (unsigned)NW / U);
    if (g >= NW) g = NW - 1;
    while (g + 1 < NW && attw_lo(U, g + 1, NW) <= u) ++g;
    while (g > 0 && attw_lo(U, g, NW) > u) --g;
    return g;
}
// units of a key whose sequence had `rows` rows when the launch began: its prefix blocks and the tail
__device__ __forceinline__ int attw_units(int rows) { return ((rows + 31) >> 5) + 1; }

// The split of the batch's units over the warps; the same for every step of a launch.
struct AttwPlan {
    unsigned U;     // units of the batch
    int NW;         // warps that take part (global warp numbers [0, NW))
};
__device__ __forceinline__ AttwPlan attw_plan(const int* pos0, int B, int HG, int NW) {
    AttwPlan pl;
    pl.U = 0;
    bool uniform = true;
    const int nb_first = attw_units(__ldg(pos0));
    for (int b = 0; b < B; ++b) {
        const int nbb = attw_units(__ldg(pos0 + b));
        pl.U += (unsigned)HG * (unsigned)nbb;
        uniform = uniform && nbb == nb_first;
    }
    // When every key has the same number of units and there are at least as many warps as keys, use a whole
    // number of warps per key: the ranges then start on key boundaries and (with one warp per key) nothing is
    // published or merged.  Otherwise all warps take equal ranges of the unit list.
    const int nkeys = B * HG;
    pl.NW = (uniform && nkeys <= NW) ? nkeys * (NW / nkeys) : NW;
    return pl;
}
__device__ __forceinline__ void attw_range(const AttwPlan& pl, int gw, unsigned& u0, unsigned& u1) {
    u0 = u1 = 0;
    if (gw >= pl.NW) return;
    u0 = attw_lo(pl.U, gw, pl.NW);
    u1 = attw_lo(pl.U, gw + 1, pl.NW);
}

// Walks a warp's units in order: what the producer thread needs to know about each of them.
struct AttwCursor {
    int b, hg, j, nb, rows;     // sequence, key of the sequence, unit of the key; units per key and prefix rows of b
    unsigned left;              // units still to come, this one included
};
__device__ __forceinline__ void attw_cursor_init(AttwCursor& c, const int* pos0, int HG, unsigned u0, unsigned u1) {
    c.b = c.hg = c.j = c.nb = c.rows = 0;
    c.left = u1 - u0;
    if (c.left == 0) return;
    unsigned cum = 0;
    for (;; ++c.b) {
        c.rows = __ldg(pos0 + c.b);
        c.nb = attw_units(c.rows);
        if (u0 < cum + (unsigned)(HG * c.nb)) break;
        cum += (unsigned)(HG * c.nb);
    }
    c.hg = (int)((u0 - cum) / (unsigned)c.nb);
    c.j = (int)((u0 - cum) % (unsigned)c.nb);
}
__device__ __forceinline__ void attw_cursor_next(AttwCursor& c, const int* pos0, int HG) {
    if (--c.left == 0) return;
    if (++c.j == c.nb) {
        c.j = 0;
        if (++c.hg == HG) {
            c.hg = 0;
            ++c.b;
            c.rows = __ldg(pos0 + c.b);
            c.nb = attw_units(c.rows);
        }
    }
}

__device__ __forceinline__ void attw_sts16(uint32_t addr, uint4 v) {
    asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void attw_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ uint4 attw_lds16(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// fp32 result and its bf16 operand copy (with the rounding remainder in row b + lo_rows when asked for)
__device__ __forceinline__ void attw_store(const AttnWArgs& a, int b, int qw, int col, float o) {
    a.attn[(long long)b * qw + col] = o;
    const bf16 hi = __float2bfloat16_rn(o);
    a.attn_h[(long long)b * qw + col] = hi;
    if (a.lo_rows > 0) a.attn_h[(long long)(b + a.lo_rows) * qw + col] = __float2bfloat16_rn(o - __bfloat162float(hi));
}

// this lane's slice of a V row: DH/32 bf16 values in one load
template <int EPL> struct AttwVec;
template <> struct AttwVec<4> {
    typedef uint2 type;
    __device__ __forceinline__ static uint2 zero() { return make_uint2(0u, 0u); }
    __device__ __forceinline__ static uint2 lds(uint32_t addr) {
        uint2 v;
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
        return v;
    }
    __device__ __forceinline__ static void unpack(uint2 w, float (&f)[4]) {
        f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
    }
};
template <> struct AttwVec<2> {
    typedef unsigned type;
    __device__ __forceinline__ static unsigned zero() { return 0u; }
    __device__ __forceinline__ static unsigned lds(uint32_t addr) {
        unsigned v;
        asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
        return v;
    }
    __device__ __forceinline__ static void unpack(unsigned w, float (&f)[2]) { f[0] = bf16_lo(w); f[1] = bf16_hi(w); }
};

// Ring: acquire(r, addr) waits for the stage that holds this warp's r-th unit and returns its shared address
// (false: the wait was given up); release(r) hands the stage back (one lane calls it).
template <int DH, int GQ, typename Ring>
__device__ void attn_warp_phase(const AttnWArgs& a, const AttwPlan& pl, int gw, int lane, Ring& ring) {
    constexpr int LPR = DH / 8;          // lanes per cache row (16-byte slices)
    constexpr int RPI = 32 / LPR;        // rows per load instruction
    constexpr int NI = LPR;              // load instructions per 32-row block
    constexpr int EPL = DH / 32;         // output elements per lane
    constexpr int HALF = DH / 2;
    const int c = lane % LPR, hrow = lane / LPR;
    const int G = a.Hq / a.Hkv;
    const int HG = a.Hq / GQ;            // keys per sequence
    const int qw = a.Hq * DH, kvw = a.Hkv * DH;
    const unsigned U = pl.U;
    const int NW = pl.NW;
    unsigned u0, u1;
    attw_range(pl, gw, u0, u1);
    if (u0 >= u1) return;

    // locate the first unit
    int b = 0;
    unsigned cum = 0;            // first unit of sequence b
    int rows = 0, nb = 0;        // prefix rows and units per key of sequence b
    for (;; ++b) {
        rows = __ldg(a.pos0 + b);
        nb = attw_units(rows);
        if (u0 < cum + (unsigned)(HG * nb)) break;
        cum += (unsigned)(HG * nb);
    }
    int hg = (int)((u0 - cum) / nb), j = (int)((u0 - cum) % nb);

    float qf[GQ][8], cs8[8], sn8[8];
    float m_run[GQ], l_run[GQ], acc[GQ][EPL];
    bool fresh = true;           // state must be initialised for the current key
    int j_first = 0, nblk = 0;   // first block and number of blocks of the running partial

    for (unsigned u = u0; u < u1; ++u) {
        const int len = rows + a.step + 1;           // rows attended to at this step
        const int p = len - 1;                       // the new position's row
        const bool tail = j == nb - 1;               // the rows of this launch; else a prefix block in the ring
        uint32_t stage = 0;
        if (!ring.acquire(u - u0, stage)) return;
        const int slot = __ldg(a.slots + b);
        const float* qkv = a.qkv + (long long)b * a.ld;
        const int h0 = hg * GQ, kvh = h0 / G;
        bf16* Kbase = a.Kc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
        bf16* Vbase = a.Vc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
        if (fresh) {
            // rotation of this lane's slice [8c, 8c+8) at position p (the same for every head), then the slice
            // of every query head of the group, rotated and scaled
            {
                const float4* tab = (const float4*)(a.rope_tab + (long long)b * HALF + ((8 * c) & (HALF - 1)));
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const float4 t = __ldcg(tab + e2);
                    cs8[2 * e2] = t.x; sn8[2 * e2] = t.y; cs8[2 * e2 + 1] = t.z; sn8[2 * e2 + 1] = t.w;
                }
            }
            const bool lower = 8 * c < HALF;                  // this slice lies in the first half of the head
#pragma unroll
            for (int g = 0; g < GQ; ++g) {
                const float* q = qkv + (h0 + g) * DH;
                const float4 x0 = __ldcg((const float4*)(q + 8 * c)), x1 = __ldcg((const float4*)(q + 8 * c) + 1);
                const float4 y0 = __ldcg((const float4*)(q + ((8 * c) ^ HALF))), y1 = __ldcg((const float4*)(q + ((8 * c) ^ HALF)) + 1);
                const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                const float ys[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    qf[g][e] = (lower ? xs[e] * cs8[e] - ys[e] * sn8[e] : xs[e] * cs8[e] + ys[e] * sn8[e]) * a.scale;
                m_run[g] = -INFINITY;
                l_run[g] = 0.f;
#pragma unroll
                for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
            }
            j_first = j;
            nblk = 0;
            fresh = false;
        }
        const int base = tail ? rows : (j << 5);
        const int nrows = tail ? a.step + 1 : min(rows - base, 32);
        // Stage layout: K row r of the unit at r * DH, V row r at (32 + r) * DH (bf16 elements).
        if (tail) {
            // The tail's stage arrived empty.  Fill it here: the rows that earlier steps of this launch
            // appended (read from the cache), then the new position's row - K rotated and rounded to what the
            // cache will hold, V likewise - which the key that owns the KV head also appends to the cache.
            const int nold = a.step;
            for (int i = lane; i < nold * LPR; i += 32) {
                const int r = i / LPR, ch = i % LPR;
                const uint4 kk = __ldcg((const uint4*)(Kbase + (long long)(rows + r) * DH) + ch);
                const uint4 vv = __ldcg((const uint4*)(Vbase + (long long)(rows + r) * DH) + ch);
                attw_sts16(stage + (uint32_t)(r * DH * 2 + ch * 16), kk);
                attw_sts16(stage + (uint32_t)((32 + r) * DH * 2 + ch * 16), vv);
            }
            if (hrow == 0) {
                const bool lower = 8 * c < HALF;
                const float* kx = qkv + qw + kvh * DH;
                const float4 x0 = __ldcg((const float4*)(kx + 8 * c)), x1 = __ldcg((const float4*)(kx + 8 * c) + 1);
                const float4 y0 = __ldcg((const float4*)(kx + ((8 * c) ^ HALF))), y1 = __ldcg((const float4*)(kx + ((8 * c) ^ HALF)) + 1);
                const float* vx = qkv + qw + kvw + kvh * DH + 8 * c;
                const float4 v0 = __ldcg((const float4*)vx), v1 = __ldcg((const float4*)vx + 1);
                const float xs[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                const float ys[8] = {y0.x, y0.y, y0.z, y0.w, y1.x, y1.y, y1.z, y1.w};
                const float vs[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
                unsigned pk[4], pv[4];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const float kr = lower ? xs[e] * cs8[e] - ys[e] * sn8[e] : xs[e] * cs8[e] + ys[e] * sn8[e];
                    const unsigned kb = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(kr));
                    const unsigned vb = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(vs[e]));
                    if (e & 1) { pk[e >> 1] |= kb << 16; pv[e >> 1] |= vb << 16; }
                    else { pk[e >> 1] = kb; pv[e >> 1] = vb; }
                }
                const uint4 kq = make_uint4(pk[0], pk[1], pk[2], pk[3]), vq = make_uint4(pv[0], pv[1], pv[2], pv[3]);
                attw_sts16(stage + (uint32_t)(nold * DH * 2 + c * 16), kq);
                attw_sts16(stage + (uint32_t)((32 + nold) * DH * 2 + c * 16), vq);
                if ((h0 % G) == 0) {         // one key per KV head appends the row
                    *(uint4*)(Kbase + (long long)p * DH + 8 * c) = kq;
                    *(uint4*)(Vbase + (long long)p * DH + 8 * c) = vq;
                }
            }
            __syncwarp();
        }
        // The loops over the rows are kept rolled on purpose: a warp runs alone on its scheduler here, and a
        // long unrolled body would be bound by instruction fetch.
        // ---- scores: partial dot products of this lane's slice, reduced eight load instructions at a time
        float sc[GQ];            // the complete score of row (c * RPI + hrow) of the unit, one per head
#pragma unroll
        for (int g = 0; g < GQ; ++g) sc[g] = 0.f;
#pragma unroll 1
        for (int i0 = 0; i0 < NI; i0 += 8) {
            if (i0 * RPI >= nrows) break;
            uint4 kw[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int r = (i0 + t) * RPI + hrow;
                kw[t] = r < nrows ? attw_lds16(stage + (uint32_t)(r * DH + 8 * c) * 2u) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int g = 0; g < GQ; ++g) {
                float v[8];
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    const uint4 w = kw[t];
                    float s = qf[g][0] * bf16_lo(w.x);
                    s = fmaf(qf[g][1], bf16_hi(w.x), s);
                    s = fmaf(qf[g][2], bf16_lo(w.y), s);
                    s = fmaf(qf[g][3], bf16_hi(w.y), s);
                    s = fmaf(qf[g][4], bf16_lo(w.z), s);
                    s = fmaf(qf[g][5], bf16_hi(w.z), s);
                    s = fmaf(qf[g][6], bf16_lo(w.w), s);
                    v[t] = fmaf(qf[g][7], bf16_hi(w.w), s);
                }
                // transposing butterfly over the lanes of a row: afterwards v[0] is the sum for t = c & 7
#pragma unroll
                for (int off = 4; off >= 1; off >>= 1) {
                    const bool up = (c & off) != 0;
#pragma unroll
                    for (int t = 0; t < off; ++t) {
                        const float send = up ? v[t] : v[t + off];
                        const float keep = up ? v[t + off] : v[t];
                        v[t] = keep + __shfl_xor_sync(0xffffffffu, send, off);
                    }
                }
                if (LPR == 16) {
                    v[0] += __shfl_xor_sync(0xffffffffu, v[0], 8);      // the other eight lanes of the row
                    if ((c >> 3) == (i0 >> 3)) sc[g] = v[0];            // this group of eight holds instruction c
                } else {
                    sc[g] = v[0];
                }
            }
        }
        const bool ok = c * RPI + hrow < nrows;
        // ---- online softmax over the block
        float pr[GQ];
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            const float sv = ok ? sc[g] : -INFINITY;
            float mb = sv;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, o));
            const float mn = fmaxf(m_run[g], mb);           // finite: the block has at least one row
            const float corr = expf(m_run[g] - mn);
            pr[g] = ok ? expf(sv - mn) : 0.f;
            float ps = pr[g];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(0xffffffffu, ps, o);
            l_run[g] = l_run[g] * corr + ps;
            m_run[g] = mn;
#pragma unroll
            for (int e = 0; e < EPL; ++e) acc[g][e] *= corr;
        }
        // ---- PV, eight rows per turn: row r's probability sits in lane (r % RPI) * LPR + r / RPI
        typedef typename AttwVec<EPL>::type vec_t;
#pragma unroll 1
        for (int r0 = 0; r0 < nrows; r0 += 8) {
            vec_t vw[8];
#pragma unroll
            for (int t = 0; t < 8; ++t)
                vw[t] = r0 + t < nrows ? AttwVec<EPL>::lds(stage + (uint32_t)((32 + r0 + t) * DH + lane * EPL) * 2u)
                                       : AttwVec<EPL>::zero();
#pragma unroll
            for (int t = 0; t < 8; ++t) {
                const int r = r0 + t;
                float vf[EPL];
                AttwVec<EPL>::unpack(vw[t], vf);
                const int src = (r % RPI) * LPR + r / RPI;
#pragma unroll
                for (int g = 0; g < GQ; ++g) {
                    const float pj = __shfl_sync(0xffffffffu, pr[g], src);          // 0 for rows beyond the block
#pragma unroll
                    for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(pj, vf[e], acc[g][e]);
                }
            }
        }
        if (tail) attw_fence_async_smem();       // this warp wrote the stage; the next copy into it is asynchronous
        ++nblk;
        __syncwarp();
        if (lane == 0) ring.release(u - u0);

        // ---- next unit; flush when the key changes or this warp's range ends
        const int b_cur = b, hg_cur = hg, nb_cur = nb;
        const unsigned k0 = cum + (unsigned)(hg * nb);               // first unit of the current key
        bool key_ends = false;
        if (++j == nb) {
            j = 0;
            key_ends = true;
            if (++hg == HG) {
                hg = 0;
                cum += (unsigned)(HG * nb);
                ++b;
                if (b < a.B) {
                    rows = __ldg(a.pos0 + b);
                    nb = attw_units(rows);
                }
            }
        }
        if (!key_ends && u + 1 < u1) continue;
        fresh = true;
        if (nblk == nb_cur) {
            // the whole key was done here: write the result
#pragma unroll
            for (int g = 0; g < GQ; ++g)
#pragma unroll
                for (int e = 0; e < EPL; ++e)
                    attw_store(a, b_cur, qw, (hg_cur * GQ + g) * DH + lane * EPL + e, acc[g][e] / l_run[g]);
            continue;
        }
        // publish the partial in the slot of its first block
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            const long long pi = ((long long)b_cur * a.Hq + hg_cur * GQ + g) * a.nslot + j_first;
#pragma unroll
            for (int e = 0; e < EPL; ++e) __stcg(a.part_acc + pi * DH + lane * EPL + e, acc[g][e]);
            if (lane == 0) {
                __stcg(a.part_ml + pi * 2, m_run[g]);
                __stcg(a.part_ml + pi * 2 + 1, l_run[g]);
            }
        }
        __syncwarp();
        int last = 0;
        if (lane == 0) {
            int* ctr = a.counters + b_cur * HG + hg_cur;
            const int old = atom_add_acq_rel(ctr, nblk);
            last = (old + nblk == nb_cur);
            if (last) *ctr = 0;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (!last) continue;
        // merge the key's partials in block order (a partial starts where a warp's range meets the key), one
        // pass with running rescaling, all heads of the group per partial
        float M[GQ], L[GQ], A[GQ][EPL];
#pragma unroll
        for (int g = 0; g < GQ; ++g) {
            M[g] = -INFINITY;
            L[g] = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) A[g][e] = 0.f;
        }
        for (unsigned uu = k0; uu < k0 + (unsigned)nb_cur;) {
#pragma unroll
            for (int g = 0; g < GQ; ++g) {
                const long long pi = ((long long)b_cur * a.Hq + hg_cur * GQ + g) * a.nslot + (uu - k0);
                const float m = __ldcg(a.part_ml + pi * 2), l = __ldcg(a.part_ml + pi * 2 + 1);
                const float Mn = fmaxf(M[g], m);
                const float fo = expf(M[g] - Mn), fn = expf(m - Mn);
                L[g] = L[g] * fo + l * fn;
#pragma unroll
                for (int e = 0; e < EPL; ++e) A[g][e] = A[g][e] * fo + __ldcg(a.part_acc + pi * DH + lane * EPL + e) * fn;
                M[g] = Mn;
            }
            uu = attw_lo(U, attw_owner(U, NW, uu) + 1, NW);
        }
#pragma unroll
        for (int g = 0; g < GQ; ++g)
#pragma unroll
            for (int e = 0; e < EPL; ++e) attw_store(a, b_cur, qw, (hg_cur * GQ + g) * DH + lane * EPL + e, A[g][e] / L[g]);
    }
}
