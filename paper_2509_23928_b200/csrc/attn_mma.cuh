// Tensor-core variant of the warp-granular decode attention of the tensor-core chain kernel, used when several
// query heads share a KV head (a group of up to eight heads is one MMA operand).
//
// Unit of work, ring staging and the tail unit are as in attn_warp.cuh; what differs:
//   * a stage holds the block in the layout the matrix loads want (tiled copies with the 128-byte swizzle);
//   * scores and P V are mma.sync m16n8k16 (bf16 in, fp32 accumulate).  Q and the probabilities are fed as a
//     bf16 value plus the bf16 of its rounding remainder (rows g and g + 8 of the A operand), which keeps
//     about 16 mantissa bits of them;
//   * a warp works on ONE key, or one part of a key cut into parts (see AttmPlan), so it sets up Q once and
//     writes once.
#pragma once
#include "attn_warp.cuh"

// How the keys of the batch are given to the warps; the same for every step of a launch.
//   Enough warps (keys <= warps): a warp works on ONE key.  Keys of long sequences are cut into `parts`
//   consecutive runs of units, one warp each: the smallest T is found for which giving every key
//   ceil(units / T) warps fits the warps there are (T at least 2 units, at most 32 parts per key).  A warp thus
//   sets up Q once and writes once; only cut keys publish partials, merged by the warp that arrives last.
//   More keys than warps: every warp takes a run of whole keys, one after the other; nothing is merged.
struct AttmPlan {
    int T;          // units per part (keys <= warps), or 0: whole keys per warp
    int NW;         // warps that may take part (global warp numbers [0, NW))
    int nkeys;
};
__device__ __forceinline__ AttmPlan attm_plan(const int* pos0, int B, int HG, int NW) {
    AttmPlan pl;
    pl.NW = NW;
    pl.nkeys = B * HG;
    pl.T = 0;
    if (pl.nkeys > NW) return pl;
    int nbmax = 0;
    for (int b = 0; b < B; ++b) nbmax = max(nbmax, attw_units(__ldg(pos0 + b)));
    int lo = max(2, (nbmax + 31) / 32), hi = max(lo, nbmax);        // hi is feasible: one warp per key
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        int need = 0;
        for (int b = 0; b < B; ++b) need += HG * ((attw_units(__ldg(pos0 + b)) + mid - 1) / mid);
        if (need <= NW) hi = mid; else lo = mid + 1;
    }
    pl.T = lo;
    return pl;
}

// The work of one warp: keys [k0, k1) in (sequence, key) order; of the first key the units [j0, j1) (part
// `part` of `parts`), of any further key all units.
struct AttmJob {
    int k0, k1, j0, j1, part, parts;
    unsigned units;             // units in all
};
__device__ __forceinline__ AttmJob attm_job(const AttmPlan& pl, const int* pos0, int B, int HG, int gw) {
    AttmJob jb;
    jb.k0 = jb.k1 = jb.j0 = jb.j1 = jb.part = 0;
    jb.parts = 1;
    jb.units = 0;
    if (gw >= pl.NW) return jb;
    if (pl.T > 0) {
        int first = 0;          // first warp of sequence b
        for (int b = 0; b < B; ++b) {
            const int nb = attw_units(__ldg(pos0 + b));
            const int w = (nb + pl.T - 1) / pl.T;
            if (gw < first + HG * w) {
                const int local = gw - first;
                jb.k0 = b * HG + local / w;
                jb.k1 = jb.k0 + 1;
                jb.part = local % w;
                jb.parts = w;
                jb.j0 = nb * jb.part / w;
                jb.j1 = nb * (jb.part + 1) / w;
                jb.units = (unsigned)(jb.j1 - jb.j0);
                return jb;
            }
            first += HG * w;
        }
        return jb;              // a warp beyond the last key
    }
    jb.k0 = (int)((long long)pl.nkeys * gw / pl.NW);
    jb.k1 = (int)((long long)pl.nkeys * (gw + 1) / pl.NW);
    for (int k = jb.k0; k < jb.k1; ++k) jb.units += (unsigned)attw_units(__ldg(pos0 + k / HG));
    if (jb.k0 < jb.k1) jb.j1 = attw_units(__ldg(pos0 + jb.k0 / HG));
    return jb;
}

// Walks a warp's units in order: what the producer thread needs to know about each of them.
struct AttmCursor {
    int k, k1, hg, j, j1;       // key (global number), end of the job's keys, key of its sequence, unit, end of the key's units
    int nb, rows, slot;         // units per key, prefix rows and cache slot of the key's sequence
    unsigned left;              // units still to come, this one included
};
__device__ __forceinline__ void attm_cursor_init(AttmCursor& c, const AttmJob& jb, const int* pos0, const int* slots, int HG) {
    c.k = jb.k0; c.k1 = jb.k1; c.j = jb.j0; c.j1 = jb.j1; c.left = jb.units;
    c.hg = c.nb = c.rows = c.slot = 0;
    if (c.left == 0) return;
    const int b = c.k / HG;
    c.hg = c.k - b * HG;
    c.rows = __ldg(pos0 + b);
    c.nb = attw_units(c.rows);
    c.slot = __ldg(slots + b);
}
__device__ __forceinline__ void attm_cursor_next(AttmCursor& c, const int* pos0, const int* slots, int HG) {
    if (--c.left == 0) return;
    if (++c.j == c.j1) {        // next key of the job (whole keys)
        ++c.k;
        if (++c.hg == HG) {
            c.hg = 0;
            const int b = c.k / HG;
            c.rows = __ldg(pos0 + b);
            c.nb = attw_units(c.rows);
            c.slot = __ldg(slots + b);
        }
        c.j = 0;
        c.j1 = c.nb;
    }
}

// Byte offset of 16-byte chunk `ch` of row `r` in a stage's K (or V) part: sub-tiles of 64 elements (128-byte
// rows, 32 rows, 4 KB each), the chunk position within the row xor-ed with the row number (128-byte swizzle).
template <int DH>
__device__ __forceinline__ uint32_t attm_swz(int r, int ch) {
    return (uint32_t)((ch >> 3) * 4096 + r * 128 + (((ch & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ unsigned attm_pack(bf16 lo, bf16 hi) {
    return (unsigned)__bfloat16_as_ushort(lo) | ((unsigned)__bfloat16_as_ushort(hi) << 16);
}
// four 8x8 bf16 blocks from shared memory (lane l gives the address of row l % 8 of block l / 8)
__device__ __forceinline__ void attm_ldsm4(unsigned (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void attm_ldsm4t(unsigned (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A B, m16n8k16, bf16 operands, fp32 accumulation
__device__ __forceinline__ void attm_mma(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Ring: acquire(r, addr) waits for the stage that holds this warp's r-th unit and returns its shared address
// (false: the wait was given up); release(r) hands the stage back (one lane calls it).
template <int DH, int GQ, typename Ring>
__device__ void attn_mma_phase(const AttnWArgs& a, const AttmJob& jb, int lane, Ring& ring) {
    constexpr int LPR = DH / 8;          // 16-byte chunks per cache row
    constexpr int KS = DH / 16;          // 16-wide slices of the head dimension (k steps of the score MMAs)
    constexpr int NT = DH / 8;           // 8-wide column tiles of the output
    constexpr int HALF = DH / 2;
    constexpr uint32_t VOFF = 32 * DH * 2;      // V sub-tiles follow the K sub-tiles in a stage
    static_assert(GQ <= 8, "a group of query heads fills the eight hi rows of the A operand");
    const int G = a.Hq / a.Hkv;
    const int HG = a.Hq / GQ;            // keys per sequence
    const int qw = a.Hq * DH, kvw = a.Hkv * DH;
    if (jb.units == 0) return;

    // the first key of the job
    int k = jb.k0;
    int b = k / HG, hg = k - b * HG;
    int rows = __ldg(a.pos0 + b), nb = attw_units(rows);      // prefix rows and units per key of sequence b
    int j = jb.j0, j_end = jb.j1;

    // fragment coordinates of this lane in the m16n8k16 MMAs: g = row of A / C (a head), t = column pair
    const int g = lane >> 2, t = lane & 3;
    const bool head_ok = g < GQ;
    unsigned qa[KS][4];          // A fragments of Q for every 16-wide slice of the head dimension
    float o[NT][4];              // C fragments of the output: o[j][0..1] head g (hi part), o[j][2..3] its lo part
    float m_run = -INFINITY, l_run = 0.f;
    bool fresh = true;           // state must be initialised for the current key
    int nblk = 0;                // units of the current key done by this warp

    for (unsigned u = 0; u < jb.units; ++u) {
        const int len = rows + a.step + 1;           // rows attended to at this step
        const int p = len - 1;                       // the new position's row
        const bool tail = j == nb - 1;               // the rows of this launch; else a prefix block in the ring
        const int slot = __ldg(a.slots + b);
        const float* qkv = a.qkv + (long long)b * a.ld;
        const int h0 = hg * GQ, kvh = h0 / G;
        bf16* Kbase = a.Kc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
        bf16* Vbase = a.Vc + ((long long)slot * a.Hkv + kvh) * (long long)a.max_len * DH;
        if (fresh) {
            // Q of head h0 + g, rotated to position p and scaled, split into a bf16 value and the bf16 of the
            // rounding remainder (rows g and g + 8 of the A operand); heads beyond the group are zero rows
            const float* q = qkv + (h0 + (head_ok ? g : 0)) * DH;
            const float2* tab = a.rope_tab + (long long)b * HALF;
#pragma unroll
            for (int kk = 0; kk < KS; ++kk) {
#pragma unroll
                for (int hh = 0; hh < 2; ++hh) {
                    const int d0 = 16 * kk + 8 * hh + 2 * t;             // dims d0, d0 + 1
                    float r0 = 0.f, r1 = 0.f;
                    if (head_ok) {
                        const float2 x = __ldcg((const float2*)(q + d0));
                        const float2 y = __ldcg((const float2*)(q + (d0 ^ HALF)));
                        const float4 cs = __ldcg((const float4*)(tab + (d0 & (HALF - 1))));     // cos, sin, cos, sin
                        const bool lower = d0 < HALF;
                        r0 = (lower ? x.x * cs.x - y.x * cs.y : x.x * cs.x + y.x * cs.y) * a.scale;
                        r1 = (lower ? x.y * cs.z - y.y * cs.w : x.y * cs.z + y.y * cs.w) * a.scale;
                    }
                    const bf16 h0b = __float2bfloat16_rn(r0), h1b = __float2bfloat16_rn(r1);
                    const bf16 l0b = __float2bfloat16_rn(r0 - __bfloat162float(h0b)), l1b = __float2bfloat16_rn(r1 - __bfloat162float(h1b));
                    qa[kk][2 * hh] = attm_pack(h0b, h1b);
                    qa[kk][2 * hh + 1] = attm_pack(l0b, l1b);
                }
            }
#pragma unroll
            for (int jn = 0; jn < NT; ++jn) o[jn][0] = o[jn][1] = o[jn][2] = o[jn][3] = 0.f;
            m_run = -INFINITY;
            l_run = 0.f;
            nblk = 0;
            fresh = false;
        }
        uint32_t stage = 0;
        if (!ring.acquire(u, stage)) return;
        const int base = tail ? rows : (j << 5);
        const int nrows = tail ? a.step + 1 : min(rows - base, 32);
        // Stage layout (what the tiled copies of the producer leave): sub-tiles of 32 rows x 64 elements, a row
        // 128 bytes, its 16-byte chunks permuted by the row number (128-byte swizzle); K sub-tiles first, then V.
        if (tail) {
            // The tail's stage arrived empty.  Fill it here in the same layout: the rows that earlier steps of
            // this launch appended (read from the cache), then the new position's row - K rotated and rounded to
            // what the cache will hold, V likewise - which the key that owns the KV head also appends to the
            // cache.  V rows up to the next multiple of 16 are cleared (they meet zero probabilities, but must
            // be numbers).
            const int nold = a.step;
            for (int i = lane; i < nold * LPR; i += 32) {
                const int r = i / LPR, ch = i % LPR;
                const uint4 kk = __ldcg((const uint4*)(Kbase + (long long)(rows + r) * DH) + ch);
                const uint4 vv = __ldcg((const uint4*)(Vbase + (long long)(rows + r) * DH) + ch);
                attw_sts16(stage + attm_swz<DH>(r, ch), kk);
                attw_sts16(stage + VOFF + attm_swz<DH>(r, ch), vv);
            }
            const int rfill = (nrows + 15) & ~15;
            for (int i = lane; i < (rfill - nrows) * LPR; i += 32) {
                const int r = nrows + i / LPR, ch = i % LPR;
                attw_sts16(stage + VOFF + attm_swz<DH>(r, ch), make_uint4(0u, 0u, 0u, 0u));
            }
            if (lane < LPR) {
                const int c = lane;
                const bool lower = 8 * c < HALF;
                const float* kx = qkv + qw + kvh * DH;
                const float4 x0 = __ldcg((const float4*)(kx + 8 * c)), x1 = __ldcg((const float4*)(kx + 8 * c) + 1);
                const float4 y0 = __ldcg((const float4*)(kx + ((8 * c) ^ HALF))), y1 = __ldcg((const float4*)(kx + ((8 * c) ^ HALF)) + 1);
                const float* vx = qkv + qw + kvw + kvh * DH + 8 * c;
                const float4 v0 = __ldcg((const float4*)vx), v1 = __ldcg((const float4*)vx + 1);
                const float4* tab = (const float4*)(a.rope_tab + (long long)b * HALF + ((8 * c) & (HALF - 1)));
                float cs8[8], sn8[8];
#pragma unroll
                for (int e2 = 0; e2 < 4; ++e2) {
                    const float4 tt = __ldcg(tab + e2);
                    cs8[2 * e2] = tt.x; sn8[2 * e2] = tt.y; cs8[2 * e2 + 1] = tt.z; sn8[2 * e2 + 1] = tt.w;
                }
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
                attw_sts16(stage + attm_swz<DH>(nold, c), kq);
                attw_sts16(stage + VOFF + attm_swz<DH>(nold, c), vq);
                if ((h0 % G) == 0) {         // one key per KV head appends the row
                    *(uint4*)(Kbase + (long long)p * DH + 8 * c) = kq;
                    *(uint4*)(Vbase + (long long)p * DH + 8 * c) = vq;
                }
            }
            __syncwarp();
        }
        // ---- scores S[head][row] = Q K^T on the tensor cores (m16n8k16, bf16 in, fp32 out): A = Q (hi rows
        //      0..7, lo rows 8..15), B = 8 rows of K (K is stored row-major, which is what the B operand wants)
        //      All four 8-row tiles are computed, also those beyond the block (their scores are discarded): four
        //      independent accumulator chains keep the tensor pipe busy, a branch per tile would serialise them.
        float sc[4][2];          // head g, rows 8 nt + 2t, 8 nt + 2t + 1 of the unit
        {
            float c4[4][4];
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) c4[nt][0] = c4[nt][1] = c4[nt][2] = c4[nt][3] = 0.f;
#pragma unroll
            for (int kk = 0; kk < KS; kk += 2) {
                // per tile four 8x8 blocks: rows 8 nt.., 16-byte chunks 2 kk .. 2 kk + 3 (two k slices)
                unsigned kb4[4][4];
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
                    attm_ldsm4(kb4[nt], stage + attm_swz<DH>(8 * nt + (lane & 7), 2 * kk + (lane >> 3)));
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) attm_mma(c4[nt], qa[kk], kb4[nt][0], kb4[nt][1]);
#pragma unroll
                for (int nt = 0; nt < 4; ++nt) attm_mma(c4[nt], qa[kk + 1], kb4[nt][2], kb4[nt][3]);
            }
#pragma unroll
            for (int nt = 0; nt < 4; ++nt) {
                const int r0 = 8 * nt + 2 * t;
                sc[nt][0] = r0 < nrows ? c4[nt][0] + c4[nt][2] : -INFINITY;
                sc[nt][1] = r0 + 1 < nrows ? c4[nt][1] + c4[nt][3] : -INFINITY;
            }
        }
        // ---- online softmax over the block (a head's scores sit in the four lanes of a quad)
        float mb = fmaxf(fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                         fmaxf(fmaxf(sc[2][0], sc[2][1]), fmaxf(sc[3][0], sc[3][1])));
        mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 1));
        mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, 2));
        const float mn = fmaxf(m_run, mb);              // finite: the block has at least one row
        const float corr = __expf(m_run - mn);
        float ps = 0.f;
        unsigned pa[2][4];       // A fragments of P for the two 16-row slices: hi in rows 0..7, lo in rows 8..15
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) {
            const float p0 = __expf(sc[nt][0] - mn), p1 = __expf(sc[nt][1] - mn);      // 0 for rows beyond the block
            ps += p0 + p1;
            const bf16 h0b = __float2bfloat16_rn(p0), h1b = __float2bfloat16_rn(p1);
            const bf16 l0b = __float2bfloat16_rn(p0 - __bfloat162float(h0b)), l1b = __float2bfloat16_rn(p1 - __bfloat162float(h1b));
            pa[nt >> 1][2 * (nt & 1)] = attm_pack(h0b, h1b);
            pa[nt >> 1][2 * (nt & 1) + 1] = attm_pack(l0b, l1b);
        }
        ps += __shfl_xor_sync(0xffffffffu, ps, 1);
        ps += __shfl_xor_sync(0xffffffffu, ps, 2);
        l_run = l_run * corr + ps;
        m_run = mn;
#pragma unroll
        for (int jn = 0; jn < NT; ++jn) {
            o[jn][0] *= corr; o[jn][1] *= corr; o[jn][2] *= corr; o[jn][3] *= corr;
        }
        // ---- O += P V: A = P, B = 16 rows of V x 8 columns (V is row-major: the transposing matrix load)
#pragma unroll
        for (int ks = 0; ks < 2; ++ks) {
            if (16 * ks < nrows) {
#pragma unroll
                for (int jn = 0; jn < NT; jn += 2) {
                    // four 8x8 blocks: rows 16 ks .. +7 and +8 .. +15 of chunk jn, the same of chunk jn + 1
                    unsigned vb4[4];
                    attm_ldsm4t(vb4, stage + VOFF + attm_swz<DH>(16 * ks + 8 * ((lane >> 3) & 1) + (lane & 7), jn + (lane >> 4)));
                    attm_mma(o[jn], pa[ks], vb4[0], vb4[1]);
                    attm_mma(o[jn + 1], pa[ks], vb4[2], vb4[3]);
                }
            }
        }
        ++nblk;
        if (tail) attw_fence_async_smem();       // this warp wrote the stage; the next copy into it is asynchronous
        __syncwarp();
        if (lane == 0) ring.release(u);

        // ---- next unit; at the end of the key (or of this warp's part of it) the result is written
        if (++j < j_end) continue;
        const int b_cur = b, hg_cur = hg, nb_cur = nb;
        const bool cut = k == jb.k0 && jb.parts > 1;         // this key is shared with other warps
        fresh = true;
        if (++k < jb.k1) {           // next key of the job (whole keys)
            if (++hg == HG) {
                hg = 0;
                ++b;
                rows = __ldg(a.pos0 + b);
                nb = attw_units(rows);
            }
            j = 0;
            j_end = nb;
        }
        // this lane's part of the result: head hg_cur * GQ + g, elements 8 jn + 2t and the next, hi + lo parts
        const int hcol = (hg_cur * GQ + g) * DH + 2 * t;
        if (!cut) {
            // the whole key was done here: write the result
            if (head_ok) {
                const float inv = 1.f / l_run;
#pragma unroll
                for (int jn = 0; jn < NT; ++jn) {
                    attw_store(a, b_cur, qw, hcol + 8 * jn, (o[jn][0] + o[jn][2]) * inv);
                    attw_store(a, b_cur, qw, hcol + 8 * jn + 1, (o[jn][1] + o[jn][3]) * inv);
                }
            }
            continue;
        }
        // publish the partial (unnormalised) in the slot of this part
        if (head_ok) {
            const long long pi = ((long long)b_cur * a.Hq + hg_cur * GQ + g) * a.nslot + jb.part;
#pragma unroll
            for (int jn = 0; jn < NT; ++jn)
                __stcg((float2*)(a.part_acc + pi * DH + 8 * jn + 2 * t), make_float2(o[jn][0] + o[jn][2], o[jn][1] + o[jn][3]));
            if (t == 0) __stcg((float2*)(a.part_ml + pi * 2), make_float2(m_run, l_run));
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
        // merge the key's parts in order: first the largest of their maxima, then one pass over the parts whose
        // loads do not depend on each other
        if (head_ok) {
            const long long p0i = ((long long)b_cur * a.Hq + hg_cur * GQ + g) * a.nslot;
            float M = -INFINITY;
            for (int q = 0; q < jb.parts; ++q) M = fmaxf(M, __ldcg(a.part_ml + (p0i + q) * 2));
            float L = 0.f, A[NT][2];
#pragma unroll
            for (int jn = 0; jn < NT; ++jn) A[jn][0] = A[jn][1] = 0.f;
#pragma unroll 2
            for (int q = 0; q < jb.parts; ++q) {
                const float2 ml = __ldcg((const float2*)(a.part_ml + (p0i + q) * 2));
                const float fn = __expf(ml.x - M);
                L += ml.y * fn;
#pragma unroll
                for (int jn = 0; jn < NT; ++jn) {
                    const float2 x = __ldcg((const float2*)(a.part_acc + (p0i + q) * DH + 8 * jn + 2 * t));
                    A[jn][0] += x.x * fn;
                    A[jn][1] += x.y * fn;
                }
            }
            const float inv = 1.f / L;
#pragma unroll
            for (int jn = 0; jn < NT; ++jn) {
                attw_store(a, b_cur, qw, hcol + 8 * jn, A[jn][0] * inv);
                attw_store(a, b_cur, qw, hcol + 8 * jn + 1, A[jn][1] * inv);
            }
        }
    }
}
