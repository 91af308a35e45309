// Tensor-core draft-chain kernel: all k chained draft steps of up to 16 sequences in ONE cooperative
// launch, bf16 weights.
//
// One CTA per SM, 8 warps with fixed roles:
//   warp 0 (one thread)  weight producer: streams weight tiles (128 rows x 64 k, 16 KB) into a shared-memory
//                        ring with TMA (cp.async.bulk.tensor, 128-byte swizzle, mbarrier complete_tx).
//                        Weight tiles do not depend on activations, so their loads run ahead through phase
//                        and step boundaries, limited only by the ring.
//   warp 2 (one thread)  operand producer: the matching batch-operand tiles (32 rows x 64 k, 4 KB) in the
//                        same order; the first tile of a phase waits for the grid barrier before it.
//   warp 3               no role.
//   warp 1 (one thread)  issues tcgen05.mma (M = 128 weight rows, N = 32 batch columns, K = 16, four per
//                        stage), accumulating in tensor memory (two 32-column accumulators, so the next
//                        tile's MMAs overlap the previous tile's epilogue); tcgen05.commit frees stages.
//   The three single threads are the pace of the whole kernel: a stage's round trip (handed back -> copy
//   issued -> landed -> MMAs issued -> handed back) bounds the bytes in flight, so their loops hold nothing
//   that is not needed per item (one shared-memory load more per wait cost 2-4 % of a draft step).
//   warps 4-7            epilogue: tcgen05.ld (one weight row per thread, 16 batch values), then the fused
//                        output stage of the phase (residuals, RMSNorm statistics and gains, RoPE-free
//                        QKV bias, SiLU*up, LM-head argmax keys) and the bf16 operand of the next phase.
//   warps 4-7            at the start of a step: embedding gather - once the step's tokens are known, their
//                        embedding rows are copied into the dense operand buffer of the fusion FC's embedding
//                        half (a grid barrier of its own).
//   warps 4-7            between the QKV and O phases: split-KV attention over the text-only cache (one warp per
//                        scheduler: a fifth warp sharing a scheduler with another slowed both).  Its K/V
//                        blocks travel through the same ring: the rows a sequence had when the launch began
//                        do not change, so warp 0 copies them (between the QKV and the O tiles) ahead of the
//                        grid barrier, and the attention warps compute from shared memory.
//
// Work split: a phase with T row tiles and KB k-blocks is T*KB tile-k-blocks, laid out tile-major and cut
// into equal contiguous ranges, one per CTA (so every SM streams the same number of bytes whatever the
// matrix shape).  A tile that straddles CTAs is finished by whichever contributor arrives last: everyone
// writes its partial accumulator to global scratch and bumps the tile's arrival counter; the last one adds
// the partials in a fixed order (so results do not depend on timing) and runs the output stage.  Where a
// range is at least a tile long, the tile at its end is finished from an early look at the counter (the other
// contributors did their part at the start of the phase).  Nobody waits for anybody inside a phase.
//
// Batch operand: activations are rounded to bf16 for the MMA; the rounding remainder of every activation is
// fed through 16 more batch columns (rows [16, 32) of every operand buffer) and added in the output stage,
// which keeps about 16 mantissa bits of the activations for every batch size.
//
// Every wait is bounded.  A wait that runs out raises the error flag and poisons the CTA: all roles then
// run through their remaining schedule without waiting, issuing no further copies or MMAs, so that named
// barriers still pair up, tensor memory is freed and the kernel returns.
#include <cuda.h>

#include <type_traits>

#include "attn_mma.cuh"

#define TC_THREADS 256
#define TC_BK 64
#define TC_TM 128
// Batch columns of one MMA.  32: columns [0,16) take the activations rounded to bf16, columns [16,32) their
// rounding remainders, for every batch size (an MMA of this shape costs the same for 16 and for 32 columns).
// 16: the remainders use the unused columns [B, 2B), which exist only for B <= 8.
#ifndef TC_TN
#define TC_TN 32
#endif
#if TC_TN == 32
#define TC_STAGES 11
#else
#define TC_STAGES 12
#endif
#define TC_A_BYTES (TC_TM * TC_BK * 2)
#define TC_B_BYTES (TC_TN * TC_BK * 2)
#define TC_ATT_FIRST 4               // first warp that runs the attention
#define TC_ATT_WARPS (8 - TC_ATT_FIRST)
#define TC_BAR_ATT 2
#define TC_EPI_THREADS 128
#define TC_BAR_EPI 3
#define TC_TMEM_COLS (2 * TC_TN)

// instruction descriptor of tcgen05.mma kind::f16: fp32 accumulate, bf16 x bf16, both K-major, N=16, M=128
#define TC_IDESC ((1u << 4) | (1u << 7) | (1u << 10) | ((TC_TN >> 3) << 17) | ((TC_TM >> 4) << 24))

namespace {

struct TcParams {
    TcMaps maps;
    TcArgs a;
};

struct TcCtl {
    u64 full[TC_STAGES], empty[TC_STAGES], tfull[2], tempty[2];
    uint32_t tmem_base;
    unsigned issued;            // ring items the weight producer has armed so far
    int abort_flag;
    long long wait_cycles;      // limit of every wait
    int last_flag, early_flag;
    int cinfo[2][3];            // contributors of the CTA's first and last tile of the phase: first CTA, its slot bit, count
    float scale[16];
    float red[8][16];
    u64 kred[2][4][16];         // LM head: best key of each epilogue warp per sequence (two buffers, used in turn)
};

__device__ __forceinline__ uint32_t saddr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ u64 policy_evict_first() {
    u64 pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ u64 policy_evict_last() {
    u64 pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// 2-D tiled TMA load: box of the tensor map at element coordinates (x = inner, y = row)
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* map, int x, int y, uint32_t bar, u64 pol) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
        "[%0], [%1, {%2, %3}], [%4], %5;" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar), "l"(pol)
        : "memory");
}
// untiled bulk copy global -> shared (16-byte aligned addresses, size a multiple of 16 bytes)
__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const void* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
// the same for global memory only: between an acquire and tiled copies of what other CTAs wrote
__device__ __forceinline__ void fence_proxy_async_global() { asm volatile("fence.proxy.async.global;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, u64 adesc, u64 bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"((uint32_t)TC_IDESC), "r"(accumulate)
        : "memory");
}
// shared-memory matrix descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle, 8-row groups
// 1024 bytes apart
__device__ __forceinline__ u64 tc_smem_desc(uint32_t addr) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return ((u64)hi << 32) | lo;
}
__device__ __forceinline__ void tc_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
// This thread's row of an accumulator: batch columns [0,16) plus the remainder columns that go with them
// (lo_off columns further on; 0 = none), added here so that everything downstream sees 16 values.
__device__ __forceinline__ void tc_ld_acc(uint32_t taddr, float (&v)[16], int lo_off) {
    uint32_t r[16];
    tc_ld16_issue(taddr, r);
#if TC_TN == 32
    uint32_t q[16];
    tc_ld16_issue(taddr + 16, q);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + (lo_off ? __uint_as_float(q[i]) : 0.f);
#else
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]) + ((lo_off && i + lo_off < 16) ? __uint_as_float(r[(i + lo_off) & 15]) : 0.f);
#endif
}
__device__ __forceinline__ u64 ld_acquire_u64(const u64* p) {
    u64 v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add_u64(u64* p, u64 v) {
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_int(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_relaxed_int(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
// Optional time stamps (HIVIS_OPT_PHASE_TIMES): event e of step s on this CTA, in nanoseconds of the GPU's global timer.
__device__ __forceinline__ void phase_stamp(const TcArgs& a, int s, int e, int cta, int G) {
    if (a.phase_t == nullptr) return;
    u64 t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    a.phase_t[((long long)s * HIVIS_PHASE_EVENTS + e) * G + cta] = t;
}
__device__ __forceinline__ void named_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }

// ---- bounded waits -------------------------------------------------------------------------------
__device__ __forceinline__ bool poisoned(const TcCtl* ctl) { return *(volatile const int*)&ctl->abort_flag != 0; }
__device__ __forceinline__ void poison(TcCtl* ctl, int* error_flag, int code) {
    atomicCAS(error_flag, 0, code);
    *(volatile int*)&ctl->abort_flag = 1;
}
__device__ __forceinline__ bool wait_mbar(uint32_t bar, uint32_t parity, TcCtl* ctl, int* error_flag, int code) {
    if (mbar_try(bar, parity)) return true;         // the usual case costs one instruction; a completed phase is safe to use
    if (poisoned(ctl)) return false;
    const long long t0 = clock64();
    unsigned it = 0;
    while (!mbar_try(bar, parity)) {
        if ((++it & 63u) == 0u) {
            if (poisoned(ctl)) return false;
            if (ld_relaxed_int(error_flag) != 0) { *(volatile int*)&ctl->abort_flag = 1; return false; }
            if (clock64() - t0 > ctl->wait_cycles) { poison(ctl, error_flag, code); return false; }
        }
    }
    return true;
}
// Wait until the weight producer has armed ring item `idx` (absolute position).  A stage's barrier tells only
// the parity of its phase, so whoever does not consume the ring strictly in order (the attention warps; the
// MMA issuer after it stepped over attention items) first makes sure the stage is in the phase it means to
// wait for: the producer arms item idx only after item idx - TC_STAGES has been handed back.
// The count is written after the arming by the same thread with release semantics and read with acquire
// semantics (CTA scope), so a reader that sees the count finds the barrier armed.
__device__ __forceinline__ unsigned ld_acquire_cta_u32(const unsigned* p) {
    unsigned v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(saddr(p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_cta_u32(unsigned* p, unsigned v) {
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(saddr(p)), "r"(v) : "memory");
}
__device__ __forceinline__ bool wait_issued(TcCtl* ctl, unsigned idx, int* error_flag, int code) {
    if (poisoned(ctl)) return false;
    if ((int)(ld_acquire_cta_u32(&ctl->issued) - idx) > 0) return true;
    const long long t0 = clock64();
    unsigned it = 0;
    while ((int)(ld_acquire_cta_u32(&ctl->issued) - idx) <= 0) {
        if ((++it & 63u) == 0u) {
            if (poisoned(ctl)) return false;
            if (ld_relaxed_int(error_flag) != 0) { *(volatile int*)&ctl->abort_flag = 1; return false; }
            if (clock64() - t0 > ctl->wait_cycles) { poison(ctl, error_flag, code); return false; }
        }
    }
    return true;
}
// wait until the grid-wide arrival counter reaches `target`
__device__ __forceinline__ bool wait_grid(const u64* counter, u64 target, TcCtl* ctl, int* error_flag, int code) {
    if (poisoned(ctl)) return false;
    const long long t0 = clock64();
    unsigned it = 0;
    while (ld_acquire_u64(counter) < target) {
        if ((++it & 63u) == 0u) {
            if (poisoned(ctl)) return false;
            if (ld_relaxed_int(error_flag) != 0) { *(volatile int*)&ctl->abort_flag = 1; return false; }
            if (clock64() - t0 > ctl->wait_cycles) { poison(ctl, error_flag, code); return false; }
        }
    }
    return true;
}

// ---- schedule --------------------------------------------------------------------------------------
// grid barriers of one step, in order: after the embedding gather, FC, QKV, attention, O, gate/up, down, LM head
#define TC_BARS_PER_STEP 8
#define TC_SEQ_GATHER 0
#define TC_SEQ_ATTN 3
__device__ __forceinline__ int phase_seq(int p) { return p < 2 ? p + 1 : p + 2; }       // barrier a GEMM phase arrives on
__device__ __forceinline__ int need_seq(int step, int p) {                              // barrier its operand needs (-1: none)
    if (p == PH_FC) return step == 0 ? -1 : (step - 1) * TC_BARS_PER_STEP + 7;       // hidden half: the previous LM head
    return step * TC_BARS_PER_STEP + phase_seq(p) - 1;       // QKV needs FC, O needs attention, GU needs O, ...
}
struct PhaseShape {
    int nkb, ntiles;
    long long W;
};
// does this launch run the part of a step that arrives on barrier `seq`?
__device__ __forceinline__ bool seq_on(const TcArgs& a, int seq) { return seq >= a.seq_first && seq <= a.seq_last; }
__device__ __forceinline__ PhaseShape phase_shape(const TcArgs& a, int p) {
    PhaseShape s;
    s.nkb = (a.ph[p].K + TC_BK - 1) / TC_BK;
    s.ntiles = (a.ph[p].N + TC_TM - 1) / TC_TM;
    s.W = seq_on(a, phase_seq(p)) ? (long long)s.nkb * s.ntiles : 0;      // a phase outside the launch's part has no work
    return s;
}
__device__ __forceinline__ long long range_lo(long long W, int c, int G) { return W * c / G; }
// CTA whose range contains tile-k-block `idx`
__device__ __forceinline__ int owner_of(long long W, int G, long long idx) {
    int c = (int)(idx * G / W);
    if (c >= G) c = G - 1;
    while (c + 1 < G && range_lo(W, c + 1, G) <= idx) ++c;
    while (c > 0 && range_lo(W, c, G) > idx) --c;
    return c;
}

// Cursor over one CTA's tile-k-blocks through all phases and steps.  Divisions happen only when a phase is
// entered; stepping to the next k-block is a few integer instructions (the producers are single threads).
struct Cursor {
    int step, p;
    int tile, kb, left, nkb;
    bool live, entered;         // entered: this k-block is the first of its phase for this CTA
};
__device__ __forceinline__ void cursor_enter(Cursor& c, const TcArgs& a, int cta, int G) {
    // position on the first non-empty phase range at or after (step, p)
    while (c.live) {
        const PhaseShape s = phase_shape(a, c.p);
        const long long lo = range_lo(s.W, cta, G), hi = range_lo(s.W, cta + 1, G);
        c.nkb = s.nkb;
        c.left = (int)(hi - lo);
        if (c.left > 0) {
            c.tile = (int)(lo / s.nkb);
            c.kb = (int)(lo % s.nkb);
            c.entered = true;
            return;
        }
        if (++c.p == PH_COUNT) {
            c.p = 0;
            if (++c.step == a.k) c.live = false;
        }
    }
}
__device__ __forceinline__ void cursor_next(Cursor& c, const TcArgs& a, int cta, int G) {
    c.entered = false;
    if (--c.left > 0) {
        if (++c.kb == c.nkb) {
            c.kb = 0;
            ++c.tile;
        }
        return;
    }
    if (++c.p == PH_COUNT) {
        c.p = 0;
        if (++c.step == a.k) { c.live = false; return; }
    }
    cursor_enter(c, a, cta, G);
}

// after a give-up: copies already issued still land in this CTA's shared memory; give them time
__device__ __forceinline__ void drain_after_poison() {
    const long long t1 = clock64();
    while (clock64() - t1 < 4000000ll) {}
}

// ---- attention items of the ring -------------------------------------------------------------------
// The attention of a step takes its prefix blocks through the same ring as the weight tiles: between the
// QKV tiles and the O tiles of the step the weight producer issues one item per attention unit of this CTA's
// attention warps, round-robin over the warps (round r: the r-th unit of every warp that has one).  The
// attention warps consume these items; the MMA issuer and the operand producer step over them.
// Two attention bodies share this machinery: groups of query heads on one KV head (GQ > 1) take the tensor-core
// body (attn_mma.cuh: one key or part of a key per warp, swizzled stages), single heads the FMA body
// (attn_warp.cuh: equal unit ranges per warp, plain stages).
template <int GQ> struct AttSel { static constexpr bool mma = GQ > 1; };
struct TcAttInfo {
    AttwPlan pl;                    // FMA body: the split of the unit list
    AttmPlan plm;                   // tensor-core body: the plan and the work of each attention warp of this CTA
    AttmJob job[TC_ATT_WARPS];
    unsigned n[TC_ATT_WARPS];       // units of attention warp w of this CTA (global warp number w * G + cta)
    unsigned total;
};
template <int GQ>
__device__ __forceinline__ TcAttInfo tc_att_info(const TcArgs& a, int cta, int G) {
    const int HG = a.Hq / GQ;
    TcAttInfo t;
    t.total = 0;
    if constexpr (AttSel<GQ>::mma) {
        t.plm = attm_plan(a.pos0, a.B, HG, G * TC_ATT_WARPS);
        t.pl.U = 0; t.pl.NW = 0;
    } else {
        t.pl = attw_plan(a.pos0, a.B, HG, G * TC_ATT_WARPS);
        t.plm.T = 0; t.plm.NW = 0; t.plm.nkeys = 0;
    }
#pragma unroll
    for (int w = 0; w < TC_ATT_WARPS; ++w) {
        if constexpr (AttSel<GQ>::mma) {
            t.job[w] = attm_job(t.plm, a.pos0, a.B, HG, w * G + cta);
            t.n[w] = t.job[w].units;
        } else {
            unsigned u0, u1;
            attw_range(t.pl, w * G + cta, u0, u1);
            t.n[w] = u1 - u0;
        }
        t.total += t.n[w];
    }
    if (!seq_on(a, TC_SEQ_ATTN)) {
#pragma unroll
        for (int w = 0; w < TC_ATT_WARPS; ++w) {
            t.n[w] = 0;
            if constexpr (AttSel<GQ>::mma) t.job[w].units = 0;
        }
        t.total = 0;
        t.pl.U = 0;
    }
    return t;
}
__device__ __forceinline__ void ring_skip(unsigned& slot, unsigned& round, unsigned n) {
    const unsigned t = slot + n;
    round += t / TC_STAGES;
    slot = t % TC_STAGES;
}

// What an attention warp sees of the ring.
struct TcAttRing {
    TcCtl* ctl;
    int* error_flag;
    uint32_t smemA;
    unsigned base;                  // ring position of the CTA's first attention item of this step
    unsigned n[TC_ATT_WARPS];
    int w;
    __device__ __forceinline__ unsigned position(unsigned r) const {
        unsigned idx = base;
#pragma unroll
        for (int w2 = 0; w2 < TC_ATT_WARPS; ++w2) idx += (n[w2] < r ? n[w2] : r) + ((w2 < w && n[w2] > r) ? 1u : 0u);
        return idx;
    }
    __device__ __forceinline__ bool acquire(unsigned r, uint32_t& addr) {
        const unsigned idx = position(r), slot = idx % TC_STAGES, round = idx / TC_STAGES;
        addr = smemA + slot * TC_A_BYTES;
        if (!wait_issued(ctl, idx, error_flag, 15)) return false;
        return wait_mbar(saddr(&ctl->full[slot]), round & 1u, ctl, error_flag, 13);
    }
    __device__ __forceinline__ void release(unsigned r) { mbar_arrive(saddr(&ctl->empty[position(r) % TC_STAGES])); }
};

// One step's attention items (producer thread).  The prefix is not written during the launch, so these copies
// need no grid barrier.  A tail unit is an item without data.  A prefix block is
//   FMA body:         two bulk copies, its K rows to the start of the stage, its V rows behind the room of 32 K
//                     rows;
//   tensor-core body: a tiled copy per 64 elements of the head dimension, of 32 cache rows each, for K and for V
//                     (128-byte swizzle, which the matrix loads want); rows of the box beyond the prefix are
//                     fetched too and never used.
template <int GQ> using AttCursor = std::conditional_t<AttSel<GQ>::mma, AttmCursor, AttwCursor>;
template <int DH, int GQ>
__device__ bool tc_issue_attention(const TcParams& P, TcCtl* ctl, uint32_t smemA, const AttCursor<GQ> (&first)[TC_ATT_WARPS],
                                   unsigned& slot, unsigned& round, u64 pol) {
    const TcArgs& a = P.a;
    AttCursor<GQ> cur[TC_ATT_WARPS];
#pragma unroll
    for (int w = 0; w < TC_ATT_WARPS; ++w) cur[w] = first[w];
    const int HG = a.Hq / GQ, Gh = a.Hq / a.Hkv;
    bool any = true;
    while (any) {
        any = false;
#pragma unroll
        for (int w = 0; w < TC_ATT_WARPS; ++w) {
            if (cur[w].left == 0) continue;
            any = true;
            // everything the copies need is worked out before the wait for the stage: what follows the wait is on the
            // path of every item (after a give-up nobody hands stages back, so the wait itself ends the loop)
            const bool tail_item = cur[w].j == cur[w].nb - 1;
            const int kvh = cur[w].hg * GQ / Gh;
            const uint32_t dst = smemA + slot * TC_A_BYTES;
            const uint32_t bar = saddr(&ctl->full[slot]);
            int row0 = 0;
            uint32_t bytes = 0;
            long long off = 0;
            if constexpr (AttSel<GQ>::mma) {
                row0 = (cur[w].slot * a.Hkv + kvh) * a.max_len + 32 * cur[w].j;
            } else if (!tail_item) {
                const int left_rows = cur[w].rows - 32 * cur[w].j;
                bytes = (uint32_t)(left_rows < 32 ? left_rows : 32) * (DH * 2);
                off = (((long long)__ldg(a.slots + cur[w].b) * a.Hkv + kvh) * (long long)a.max_len + 32 * cur[w].j) * DH;
            }
            if (round > 0 && !wait_mbar(saddr(&ctl->empty[slot]), (round - 1) & 1u, ctl, a.error_flag, 14)) return false;
            if (tail_item) {
                mbar_arrive(bar);
            } else {
                if constexpr (AttSel<GQ>::mma) {
                    mbar_expect_tx(bar, 2 * 32 * DH * 2);
#pragma unroll
                    for (int h = 0; h < DH / 64; ++h) {
                        tma_load_2d(dst + h * 4096, &P.maps.m[TCM_K], 64 * h, row0, bar, pol);
                        tma_load_2d(dst + 32 * DH * 2 + h * 4096, &P.maps.m[TCM_V], 64 * h, row0, bar, pol);
                    }
                } else {
                    mbar_expect_tx(bar, 2 * bytes);
                    bulk_load(dst, (const bf16*)a.Kc + off, bytes, bar);
                    bulk_load(dst + 32 * DH * 2, (const bf16*)a.Vc + off, bytes, bar);
                }
            }
            if constexpr (AttSel<GQ>::mma) attm_cursor_next(cur[w], a.pos0, a.slots, HG);
            else attw_cursor_next(cur[w], a.pos0, HG);
            if (++slot == TC_STAGES) { slot = 0; ++round; }
            st_release_cta_u32(&ctl->issued, round * TC_STAGES + slot);
        }
    }
    return true;
}

// ---- producers -------------------------------------------------------------------------------------
// Weight tiles: arms the stage's barrier with the bytes of both tiles and issues the weight copy.  Runs
// ahead of the grid barriers, limited only by the ring.  Also issues the attention items of every step.
template <int DH, int GQ>
__device__ void tc_producer_w(const TcParams& P, TcCtl* ctl, uint32_t smemA, int cta, int G, const TcAttInfo& ai) {
    const TcArgs& a = P.a;
    const u64 pol_stream = policy_evict_first();
    const u64 pol_kv = policy_evict_last();       // the cache is read again at every step
    // Weights of the phases named in l2_keep are asked to stay in L2: every CTA reads the same tiles again at the next
    // draft step, and a subset of the matrices fits beside the caches.  The others stream through (evict first).
    u64 pol_w = (a.l2_keep & 1) ? pol_kv : pol_stream;
    int pol_phase = 0;
    AttCursor<GQ> first[TC_ATT_WARPS];
#pragma unroll
    for (int w = 0; w < TC_ATT_WARPS; ++w) {
        if constexpr (AttSel<GQ>::mma) {
            attm_cursor_init(first[w], ai.job[w], a.pos0, a.slots, a.Hq / GQ);
        } else {
            unsigned u0, u1;
            attw_range(ai.pl, w * G + cta, u0, u1);
            attw_cursor_init(first[w], a.pos0, a.Hq / GQ, u0, u1);
        }
    }
    Cursor c{0, 0, 0, 0, 0, 0, true, false};
    cursor_enter(c, a, cta, G);
    unsigned slot = 0, round = 0;
    int att_done = 0;               // steps whose attention items have been issued
    unsigned publish = 0;           // weight items still to be announced (those that reuse attention stages)
    bool ok = true;
    while (c.live && ok) {
        const int att_need = c.step + (c.p >= PH_O ? 1 : 0);
        while (ok && att_done < att_need) {
            ok = tc_issue_attention<DH, GQ>(P, ctl, smemA, first, slot, round, pol_kv);
            ++att_done;
            publish = TC_STAGES;
        }
        if (!ok) break;
        // (after a give-up nobody hands stages back, so the wait below ends the loop: no separate look at the flag)
        if (round > 0 && !wait_mbar(saddr(&ctl->empty[slot]), (round - 1) & 1u, ctl, a.error_flag, 3)) break;
        const uint32_t bar = saddr(&ctl->full[slot]);
        mbar_expect_tx(bar, TC_A_BYTES + TC_B_BYTES);
        if (c.p != pol_phase) {
            pol_phase = c.p;
            pol_w = ((a.l2_keep >> c.p) & 1) ? pol_kv : pol_stream;
        }
        tma_load_2d(smemA + slot * TC_A_BYTES, &P.maps.m[TCM_W + c.p], c.kb * TC_BK, c.tile * TC_TM, bar, pol_w);
        cursor_next(c, a, cta, G);
        if (++slot == TC_STAGES) { slot = 0; ++round; }
        if (publish) {
            st_release_cta_u32(&ctl->issued, round * TC_STAGES + slot);
            --publish;
        }
    }
    while (ok && !poisoned(ctl) && att_done < a.k) {
        ok = tc_issue_attention<DH, GQ>(P, ctl, smemA, first, slot, round, pol_kv);
        ++att_done;
    }
    if (poisoned(ctl)) drain_after_poison();
}

// Batch-operand tiles (one thread): same k-block order; the first tile of a phase waits for the grid barrier
// after which the operand is complete.  The embedding half of the fusion FC reads the rows that the gather
// of this step copied out of the embedding table, and waits for that barrier.
__device__ void tc_producer_x(const TcParams& P, TcCtl* ctl, uint32_t smemB, int cta, int G, unsigned att_items) {
    const TcArgs& a = P.a;
    const u64 pol_x = policy_evict_last();
    Cursor c{0, 0, 0, 0, 0, 0, true, false};
    cursor_enter(c, a, cta, G);
    unsigned slot = 0, round = 0;
    const int dkb = a.d / TC_BK;
    int map_idx = TCM_X_FEAT;
    int gathered_step = -1;
    int att_done = 0;
    while (c.live) {
        for (const int att_need = c.step + (c.p >= PH_O ? 1 : 0); att_done < att_need; ++att_done)
            ring_skip(slot, round, att_items);          // the attention items between the QKV and O tiles
        if (c.entered) {
            const int need = need_seq(c.step, c.p);
            map_idx = c.p == PH_QKV ? TCM_X_XQ : c.p == PH_O ? TCM_X_ATTN : c.p == PH_GU ? TCM_X_XM
                    : c.p == PH_DOWN ? TCM_X_ACT : TCM_X_FEAT;
            // the descriptor of the phase's operand is asked for while the barrier is still awaited
            prefetch_tensormap(&P.maps.m[map_idx]);
            if (need >= 0) {
                if (!wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)(need + 1), ctl, a.error_flag, 9)) break;
                // other CTAs wrote the operand through the generic proxy; TMA reads through the async proxy
                fence_proxy_async_global();
            }
            phase_stamp(a, c.step, 8 + c.p, cta, G);
        }
        const bool emb = c.p == PH_FC && c.kb >= dkb;
        if (emb && gathered_step != c.step) {
            if (!wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)(c.step * TC_BARS_PER_STEP + TC_SEQ_GATHER + 1), ctl,
                           a.error_flag, 11))
                break;
            fence_proxy_async_global();
            gathered_step = c.step;
        }
        if (round > 0 && !wait_mbar(saddr(&ctl->empty[slot]), (round - 1) & 1u, ctl, a.error_flag, 10)) break;
        const uint32_t bar = saddr(&ctl->full[slot]);
        const uint32_t dst = smemB + slot * TC_B_BYTES;
        if (emb) tma_load_2d(dst, &P.maps.m[TCM_X_EMB], (c.kb - dkb) * TC_BK, 0, bar, pol_x);
        else tma_load_2d(dst, &P.maps.m[map_idx], c.kb * TC_BK, 0, bar, pol_x);
        cursor_next(c, a, cta, G);
        if (++slot == TC_STAGES) { slot = 0; ++round; }
    }
    if (poisoned(ctl)) drain_after_poison();
}

// Embedding gather of step s (the four epilogue warps of every CTA, before they turn to the fusion FC): once the
// previous LM head is complete the chosen tokens are known; their embedding rows are copied into the dense operand
// buffer that the fusion FC reads.  Step 0's rows were copied by the set-up kernel.  Arrives on the gather barrier
// of the step.
__device__ void tc_gather(const TcParams& P, TcCtl* ctl, int s, int cta, int G, int etid) {
    const TcArgs& a = P.a;
    if (!seq_on(a, TC_SEQ_GATHER)) return;
    if (seq_on(a, TC_SEQ_ATTN)) {
        // (cos, sin) of every sequence's new position at this step, for the attention of this step; the two
        // halves of the table alternate between steps, since CTAs still in the previous attention read the other
        const int half = a.dh >> 1;
        float2* tab = a.rope_tab + (long long)(s & 1) * 16 * half;
        for (int i = cta * TC_EPI_THREADS + etid; i < a.B * half; i += G * TC_EPI_THREADS) {
            const int b = i / half, f = i - b * half;
            float cs, sn;
            rope_cs(__ldg(a.pos0 + b) + s, a.inv_freq[f], cs, sn);
            __stcg(tab + (long long)b * half + f, make_float2(cs, sn));
        }
    }
    if (s > 0) {
        if (etid == 0)
            wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)((s - 1) * TC_BARS_PER_STEP + 8), ctl, a.error_flag, 12);
        named_sync(TC_BAR_EPI, TC_EPI_THREADS);
        if (!poisoned(ctl)) {
            const int upr = a.d >> 3;                    // 16-byte units per row
            const int total = a.B * upr;
            for (int i = cta * TC_EPI_THREADS + etid; i < total; i += G * TC_EPI_THREADS) {
                const int b = i / upr, off = i - b * upr;
                int id = a.forced ? __ldcg(a.forced + (long long)b * a.k + (s - 1))
                                  : key_index(__ldcg(a.keys + (long long)b * a.key_stride + (s - 1)));
                id = checked_token(id, a.V, a.id_flag);
                const uint4 w = ld_stream((const uint4*)(a.embed + (long long)id * a.d) + off);
                __stcg((uint4*)(a.xe_h + (long long)b * a.d) + off, w);
            }
        }
    }
    named_sync(TC_BAR_EPI, TC_EPI_THREADS);
    if (etid == 0) {
        phase_stamp(a, s, TC_SEQ_GATHER, cta, G);
        red_release_add_u64(a.bar_counter, 1ull);
    }
}

// ---- MMA issuer ----------------------------------------------------------------------------------
__device__ void tc_mma_issuer(const TcParams& P, TcCtl* ctl, uint32_t smemA, uint32_t smemB, int cta, int G,
                              unsigned att_items) {
    const TcArgs& a = P.a;
    const uint32_t tmem = ctl->tmem_base;
    unsigned seg_cnt = 0, slot = 0, round = 0;
    unsigned check = 0;         // items whose stage last held an attention item: see wait_issued
    for (int s = 0; s < a.k; ++s)
        for (int p = 0; p < PH_COUNT; ++p) {
            const PhaseShape sh = phase_shape(a, p);
            const long long lo = range_lo(sh.W, cta, G), hi = range_lo(sh.W, cta + 1, G);
            int left = (int)(hi - lo);
            int kb0 = left > 0 ? (int)(lo % sh.nkb) : 0;
            if (p == PH_O && att_items > 0) {                       // the attention items of this step
                ring_skip(slot, round, att_items);
                check = TC_STAGES;
            }
            while (left > 0) {
                const int n = left < sh.nkb - kb0 ? left : sh.nkb - kb0;
                const unsigned acc = seg_cnt & 1u, use = seg_cnt >> 1;
                if (use > 0) wait_mbar(saddr(&ctl->tempty[acc]), (use - 1) & 1u, ctl, a.error_flag, 4);
                tc_fence_after();
                for (int j = 0; j < n; ++j) {
                    bool ok = true;
                    if (check) {
                        ok = wait_issued(ctl, round * TC_STAGES + slot, a.error_flag, 16);
                        --check;
                    }
                    ok = ok && wait_mbar(saddr(&ctl->full[slot]), round & 1u, ctl, a.error_flag, 5);
                    if (ok) {
                        tc_fence_after();
                        const u64 ad = tc_smem_desc(smemA + slot * TC_A_BYTES);
                        const u64 bd = tc_smem_desc(smemB + slot * TC_B_BYTES);
#pragma unroll
                        for (int kk = 0; kk < TC_BK / 16; ++kk)
                            tc_mma(tmem + acc * TC_TN, ad + (u64)(kk * 2), bd + (u64)(kk * 2), (j > 0 || kk > 0) ? 1u : 0u);
                        tc_commit(saddr(&ctl->empty[slot]));
                    }
                    if (++slot == TC_STAGES) { slot = 0; ++round; }
                }
                if (!poisoned(ctl)) tc_commit(saddr(&ctl->tfull[acc]));
                ++seg_cnt;
                left -= n;
                kb0 = 0;
            }
        }
}

// ---- output stages ---------------------------------------------------------------------------------
// Transposing butterfly: every lane holds 16 values (one per batch column); afterwards lane L holds the
// reduction over all 32 lanes of column warp_col16(L) (lanes L and L^1 hold the same column).  16 shuffles
// instead of 16 x 5, and they are independent of each other.
__device__ __forceinline__ int warp_col16(int lane) {
    return 8 * ((lane >> 4) & 1) + 4 * ((lane >> 3) & 1) + 2 * ((lane >> 2) & 1) + ((lane >> 1) & 1);
}
template <typename T, typename Op>
__device__ __forceinline__ T warp_reduce16(T (&v)[16], int lane, Op op) {
#pragma unroll
    for (int off = 16, n = 8; off >= 2; off >>= 1, n >>= 1) {
        const bool up = (lane & off) != 0;
#pragma unroll
        for (int t = 0; t < n; ++t) {
            const T send = up ? v[t] : v[t + n];
            const T keep = up ? v[t + n] : v[t];
            v[t] = op(keep, __shfl_xor_sync(0xffffffffu, send, off));
        }
    }
    return op(v[0], __shfl_xor_sync(0xffffffffu, v[0], 1));
}
struct OpAdd { __device__ __forceinline__ float operator()(float x, float y) const { return x + y; } };
struct OpMaxU64 { __device__ __forceinline__ u64 operator()(u64 x, u64 y) const { return x > y ? x : y; } };

__device__ __forceinline__ void store_operand(bf16* buf, int width, int b, int col, float x, int lo_rows) {
    const bf16 hi = __float2bfloat16_rn(x);
    buf[(long long)b * width + col] = hi;
    if (lo_rows > 0) buf[(long long)(b + lo_rows) * width + col] = __float2bfloat16_rn(x - __bfloat162float(hi));
}

// per-sequence scale 1/rms recovered from the partial sums of squares of the producing phase
__device__ __forceinline__ void epi_compute_scales(const TcArgs& a, TcCtl* ctl, const float* ssq, int etid) {
    const int entries = ((a.d + TC_TM - 1) / TC_TM) * 4;
    const int b = etid & 15, part = etid >> 4;
    float t = 0.f;
    for (int i = part; i < entries; i += 8) t += __ldcg(ssq + (long long)i * 16 + b);
    ctl->red[part][b] = t;
    named_sync(TC_BAR_EPI, TC_EPI_THREADS);
    if (etid < 16) {
        float tot = 0.f;
#pragma unroll
        for (int q = 0; q < 8; ++q) tot += ctl->red[q][etid];
        ctl->scale[etid] = rsqrtf(tot / (float)a.d + a.eps);
    }
    named_sync(TC_BAR_EPI, TC_EPI_THREADS);
}

// What the output stage of a tile adds to or multiplies with the accumulators: requested before the tile's
// accumulator is waited for, so that these round trips to L2 are over when it arrives.  Everything read here
// was complete before the phase began (residual rows and gains are constants; u is written by the FC phase and
// read in the O phase, y by the O phase and read in the down phase).
struct EpiPre {
    float add[16];      // per sequence: the residual stream the result is added to (FC: the step's residual row)
    float g;            // RMSNorm gain of the row (FC, O) or the QKV bias
};
// SMP: the launch draws its tokens (a kernel variant of its own: the greedy output stage stays as it is)
template <bool SMP>
__device__ __forceinline__ void epi_preload(const TcArgs& a, int p, int s, int tile, int w4, int lane, EpiPre& pre) {
    const int N = a.ph[p].N;
    const int row = tile * TC_TM + w4 * 32 + lane;
    const bool rok = row < N;
    pre.g = 0.f;
#pragma unroll
    for (int b = 0; b < 16; ++b) pre.add[b] = 0.f;
    if (!rok) return;
    if (p == PH_FC) {
        pre.g = __bfloat162float(a.norm1[row]);
        const float add0 = a.rho ? a.rho[(long long)(s < a.n_resid - 1 ? s : a.n_resid - 1) * a.d + row] : 0.f;
#pragma unroll
        for (int b = 0; b < 16; ++b) pre.add[b] = add0;
    } else if (p == PH_O) {
        pre.g = __bfloat162float(a.norm2[row]);
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (b < a.B) pre.add[b] = __ldcg(a.u + (long long)b * N + row);
    } else if (p == PH_DOWN) {
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (b < a.B) pre.add[b] = __ldcg(a.y + (long long)b * N + row);
    } else if (p == PH_QKV) {
        pre.g = a.bqkv ? __bfloat162float(a.bqkv[row]) : 0.f;
    } else if (SMP && p == PH_LM) {
        // the uniform numbers of the row's token, one per sequence (the noise is added in the output stage)
#pragma unroll
        for (int b = 0; b < 16; ++b)
            if (b < a.B) pre.add[b] = __ldg(a.gumbel_u + ((long long)b * a.k + s) * N + row);
    }
}

template <bool SMP>
__device__ __forceinline__ void epi_output(const TcArgs& a, TcCtl* ctl, int p, int s, int tile, const float (&v)[16], const EpiPre& pre,
                           unsigned& lm_calls, int w4, int lane) {
    const int N = a.ph[p].N;
    const int row = tile * TC_TM + w4 * 32 + lane;
    const bool rok = row < N;
    const int B = a.B;
    const int lo_rows = a.lo;
    float val[16];
#pragma unroll
    for (int b = 0; b < 16; ++b) val[b] = b < B ? v[b] : 0.f;

    if (p == PH_FC || p == PH_O) {
        float* outf = p == PH_FC ? a.u : a.y;
        bf16* outh = p == PH_FC ? a.xq_h : a.xm_h;
        float* ssq = p == PH_FC ? a.ssq1 : a.ssq2;
        float sq[16];
#pragma unroll
        for (int b = 0; b < 16; ++b) {
            float r = 0.f;
            if (rok && b < B) {
                r = val[b] + pre.add[b];
                outf[(long long)b * N + row] = r;
                store_operand(outh, N, b, row, pre.g * r, lo_rows);
            }
            sq[b] = r * r;
        }
        const float tot = warp_reduce16(sq, lane, OpAdd());
        const int col = warp_col16(lane);
        if ((lane & 1) == 0 && col < B) ssq[(long long)(tile * 4 + w4) * 16 + col] = tot;
    } else if (p == PH_QKV) {
        if (rok) {
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                if (b >= B) break;
                a.qkv[(long long)b * N + row] = val[b] * ctl->scale[b] + pre.g;
            }
        }
    } else if (p == PH_GU) {
        // Even rows are gate_i, odd rows up_i (i = row / 2).  Of every pair of sequences (2q, 2q + 1) the even
        // lane finishes 2q and the odd lane 2q + 1: each sends the neighbour the value the neighbour needs and
        // computes one SiLU(gate) * up per pair, without a branch, so that the eight of them overlap.
        const int F = N >> 1;
        const bool odd = (lane & 1) != 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float m0 = val[2 * q] * ctl->scale[2 * q], m1 = val[2 * q + 1] * ctl->scale[2 * q + 1];
            const float recv = __shfl_xor_sync(0xffffffffu, odd ? m0 : m1, 1);
            const float gate = odd ? recv : m0, up = odd ? m1 : recv;
            const float act = __fdividef(gate, 1.f + __expf(-gate)) * up;
            const int b = 2 * q + (odd ? 1 : 0);
            if (rok && b < B) store_operand(a.act_h, F, b, row >> 1, act, lo_rows);
        }
    } else if (p == PH_DOWN) {
        if (rok) {
#pragma unroll
            for (int b = 0; b < 16; ++b) {
                if (b >= B) break;
                const float r = pre.add[b] + val[b];
                a.feat[(long long)b * N + row] = r;
                store_operand(a.feat_h, N, b, row, r, lo_rows);
            }
        }
    } else {   // PH_LM
        u64 keys[16];
#pragma unroll
        for (int b = 0; b < 16; ++b) {
            keys[b] = 0ull;
            if (rok && b < B) {
                if (a.logits_out) a.logits_out[((long long)b * a.k + s) * a.V + row] = val[b];
                keys[b] = pack_key(SMP ? gumbel_perturbed(val[b], a.inv_t, pre.add[b]) : val[b], row);
            }
        }
        // best key per sequence: over the warp, then over the four warps through shared memory, so that one
        // atomic per sequence and tile reaches the (much contended) global keys
        const u64 best = warp_reduce16(keys, lane, OpMaxU64());
        const int col = warp_col16(lane);
        u64 (*kred)[16] = ctl->kred[lm_calls & 1u];
        ++lm_calls;
        if ((lane & 1) == 0) kred[w4][col] = best;
        named_sync(TC_BAR_EPI, TC_EPI_THREADS);
        const int etid = w4 * 32 + lane;
        if (etid < B) {
            u64 m = kred[0][etid];
#pragma unroll
            for (int w = 1; w < 4; ++w) m = kred[w][etid] > m ? kred[w][etid] : m;
            if (m) atomicMax(a.keys + (long long)etid * a.key_stride + s, m);
        }
    }
}

// ---- epilogue warps: GEMM phases -------------------------------------------------------------------
// Sum of the partial accumulators of contributors i = from, from-1, ..., to of a shared tile, folded from the
// right: acc = c_i + acc.  Up to TC_FOLD contributors' loads are in flight together (the phases with few row
// tiles have five or six contributors per tile, all finishing at the same moment: one round trip, not three).
#define TC_FOLD 5
__device__ __forceinline__ void fold_partials(const TcArgs& a, float (&acc)[16], int cf, int fs, int from, int to, int etid) {
    const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
    for (int i0 = from; i0 >= to; i0 -= TC_FOLD) {
        float4 t[TC_FOLD][4];
#pragma unroll
        for (int q = 0; q < TC_FOLD; ++q) {
            const int i = i0 - q;
            const bool on = i >= to;
            const float4* src = (const float4*)(a.partial + (long long)((cf + (on ? i : to)) * 2 + (i == 0 ? fs : 0)) * (16 * TC_TM)) + etid * 4;
#pragma unroll
            for (int r = 0; r < 4; ++r) t[q][r] = on ? __ldcg(src + r) : z4;
        }
#pragma unroll
        for (int q = 0; q < TC_FOLD; ++q) {
            if (i0 - q < to) break;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                acc[4 * r] = t[q][r].x + acc[4 * r];
                acc[4 * r + 1] = t[q][r].y + acc[4 * r + 1];
                acc[4 * r + 2] = t[q][r].z + acc[4 * r + 2];
                acc[4 * r + 3] = t[q][r].w + acc[4 * r + 3];
            }
        }
    }
}

// Runs phase p of step s for this CTA's range and arrives on the phase's grid barrier.
//
// A tile that this CTA shares with others is the sum of its contributors' partial accumulators, always added
// in the same order (from the last contributor down to the first), so the result does not depend on who
// finishes the tile.  Usually a contributor stores its partial, counts itself on the tile's arrival counter
// and, if it was the last, adds the others' partials to its own.  When this CTA's range is at least a tile
// long, the other contributors of the tile at the END of its range finished that tile long ago (it was the
// first thing they did in the phase): the counter is looked at while the MMAs of the segment still run, and if
// everybody else has arrived their partials are summed right then; once the accumulator is ready the tile is
// finished without the store, the fence, the atomic and the loads on the critical path.
// (inlined at its six call sites, so that every phase gets an output stage of its own)
template <bool SMP>
__device__ __forceinline__ void tc_epilogue_phase(const TcParams& P, TcCtl* ctl, int s, int p, unsigned& seg_cnt, int cta, int G,
                                  int w4, int lane) {
    const TcArgs& a = P.a;
    if (!seq_on(a, phase_seq(p))) return;
    const int etid = w4 * 32 + lane;
    const PhaseShape sh = phase_shape(a, p);
    const long long lo = range_lo(sh.W, cta, G), hi = range_lo(sh.W, cta + 1, G);
    long long idx = lo;
    unsigned lm_calls = 0;
    bool need_scale = (p == PH_QKV || p == PH_GU);
    const bool big = sh.W >= G;        // every CTA has work: the contributors of a tile are consecutive CTAs
    // Contributors of the (at most two) tiles this CTA shares with others, worked out while the first
    // accumulator is still being computed: first contributor, its slot bit, number of contributors.
    if (etid == 0 && lo < hi && big) {
        const long long tl[2] = {lo / sh.nkb, (hi - 1) / sh.nkb};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const long long t0 = tl[q] * sh.nkb;
            const int cf = owner_of(sh.W, G, t0);
            ctl->cinfo[q][0] = cf;
            ctl->cinfo[q][1] = t0 == range_lo(sh.W, cf, G) ? 0 : 1;
            ctl->cinfo[q][2] = owner_of(sh.W, G, t0 + sh.nkb - 1) - cf + 1;
        }
    }
    if (lo < hi && big) named_sync(TC_BAR_EPI, TC_EPI_THREADS);
    if (need_scale && lo < hi) {
        // The RMSNorm scale of this phase's operand: wait here for the phase that produced it (rather than for
        // the first accumulator, which for a short range is also the last: the sums would be fetched in the tail)
        if (etid == 0) wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)(need_seq(s, p) + 1), ctl, a.error_flag, 18);
        named_sync(TC_BAR_EPI, TC_EPI_THREADS);
        epi_compute_scales(a, ctl, p == PH_QKV ? a.ssq1 : a.ssq2, etid);
        need_scale = false;
    }
    const int tile_first = (int)(lo / sh.nkb);
    while (idx < hi) {
        const int tile = (int)(idx / sh.nkb), kb0 = (int)(idx % sh.nkb);
        const int n = (int)((hi - idx) < (long long)(sh.nkb - kb0) ? (hi - idx) : (long long)(sh.nkb - kb0));
        const bool shared = !(kb0 == 0 && n == sh.nkb);
        int cf = 0, fs = 0, nc = 0;
        if (shared && big) {
            const int q = tile == tile_first ? 0 : 1;
            cf = ctl->cinfo[q][0]; fs = ctl->cinfo[q][1]; nc = ctl->cinfo[q][2];
        }
        const int me = cta - cf;            // this CTA's place among the contributors (big phases)
        EpiPre pre;
        epi_preload<SMP>(a, p, s, tile, w4, lane, pre);
        // ---- while the MMAs of the segment run: the early look at the arrival counter
        bool early = false;
        float others[16];
#pragma unroll
        for (int c = 0; c < 16; ++c) others[c] = 0.f;
        if (shared && big && idx != lo && hi - lo >= sh.nkb) {
            if (etid == 0) {
                const int seen = ld_acquire_int(a.tile_ctr + tile);
                ctl->early_flag = seen == nc - 1;
            }
            named_sync(TC_BAR_EPI, TC_EPI_THREADS);
            early = ctl->early_flag != 0;
            if (early) fold_partials(a, others, cf, fs, nc - 1, me + 1, etid);
        }
        const unsigned acc = seg_cnt & 1u;
        wait_mbar(saddr(&ctl->tfull[acc]), (seg_cnt >> 1) & 1u, ctl, a.error_flag, 6);
        if (etid == 0 && idx + n == hi) phase_stamp(a, s, 14 + p, cta, G);
        tc_fence_after();
        float v[16];
        tc_ld_acc(ctl->tmem_base + ((uint32_t)(w4 * 32) << 16) + acc * TC_TN, v, a.lo);
        tc_fence_before();
        mbar_arrive(saddr(&ctl->tempty[acc]));
        ++seg_cnt;
        if (need_scale) {       // the operand of this phase has arrived, so the producing phase is complete
            epi_compute_scales(a, ctl, p == PH_QKV ? a.ssq1 : a.ssq2, etid);
            need_scale = false;
        }
        bool finish = true;
        if (shared && early) {
#pragma unroll
            for (int c = 0; c < 16; ++c) v[c] += others[c];
            fold_partials(a, v, cf, fs, me - 1, 0, etid);
            if (etid == 0) a.tile_ctr[tile] = 0;        // nobody else will come: ready for the tile's next use
        } else if (shared) {
            // publish the partial accumulator ([row][16 columns], 64 bytes per thread); the last arriver
            // finishes the tile
            float4* mine = (float4*)(a.partial + (long long)(cta * 2 + (idx == lo ? 0 : 1)) * (16 * TC_TM)) + etid * 4;
#pragma unroll
            for (int q = 0; q < 4; ++q) __stcg(mine + q, make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]));
            named_sync(TC_BAR_EPI, TC_EPI_THREADS);
            if (etid == 0) {
                if (!big) {
                    // contributors = the CTAs whose (non-empty) ranges meet this tile, in range order
                    const long long t0 = (long long)tile * sh.nkb;
                    for (long long i = t0; i < t0 + sh.nkb; ++nc) i = range_lo(sh.W, owner_of(sh.W, G, i) + 1, G);
                }
                // release: the CTA's partial (ordered before by the barrier) is visible first; acquire: so are
                // the partials of those that arrived before
                const int old = atom_add_acq_rel(a.tile_ctr + tile, 1);
                const int last = old == nc - 1;
                if (last) a.tile_ctr[tile] = 0;
                ctl->last_flag = last;
            }
            named_sync(TC_BAR_EPI, TC_EPI_THREADS);
            finish = ctl->last_flag != 0;
            if (finish) {
                if (big) {
                    fold_partials(a, others, cf, fs, nc - 1, me + 1, etid);
#pragma unroll
                    for (int c = 0; c < 16; ++c) v[c] += others[c];
                    fold_partials(a, v, cf, fs, me - 1, 0, etid);
                } else {
                    // few tile-k-blocks (tiny shapes): contributors in range order, all read back
#pragma unroll
                    for (int c = 0; c < 16; ++c) v[c] = 0.f;
                    const long long t0 = (long long)tile * sh.nkb;
                    for (long long i = t0; i < t0 + sh.nkb;) {
                        const int cc = owner_of(sh.W, G, i);
                        const float4* src = (const float4*)(a.partial + (long long)(cc * 2 + (i == range_lo(sh.W, cc, G) ? 0 : 1)) * (16 * TC_TM)) + etid * 4;
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const float4 t = __ldcg(src + q);
                            v[4 * q] += t.x; v[4 * q + 1] += t.y; v[4 * q + 2] += t.z; v[4 * q + 3] += t.w;
                        }
                        i = range_lo(sh.W, cc + 1, G);
                    }
                }
            }
            named_sync(TC_BAR_EPI, TC_EPI_THREADS);      // last_flag may be rewritten by the next segment
        }
        if (finish) epi_output<SMP>(a, ctl, p, s, tile, v, pre, lm_calls, w4, lane);
        idx += n;
    }
    // This CTA's part of the phase is done: arrive on the grid barrier.  All arrivals are counted in one
    // counter, so a CTA may arrive for this phase only once the barrier before it is complete.  With work in
    // the phase that is implied (its operand tiles were loaded after that barrier); without work, wait for it.
    named_sync(TC_BAR_EPI, TC_EPI_THREADS);
    if (etid == 0) {
        // (the FC phase follows the gather barrier of its step, which its hidden-half operand does not imply)
        const int need = p == PH_FC ? s * TC_BARS_PER_STEP + TC_SEQ_GATHER : need_seq(s, p);
        if ((lo == hi || p == PH_FC) && need >= 0)
            wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)(need + 1), ctl, a.error_flag, 8);
        phase_stamp(a, s, phase_seq(p), cta, G);
        red_release_add_u64(a.bar_counter, 1ull);
    }
    // Without work in the phase nothing but the wait above tells this CTA that the earlier phases are complete:
    // hold the other epilogue threads until it is over (they read those phases' results early in the next one).
    if (lo == hi) named_sync(TC_BAR_EPI, TC_EPI_THREADS);
}

}  // namespace

template <int DH, int GQ, bool SMP>
__global__ void __launch_bounds__(TC_THREADS, 1) tc_chain_kernel(const __grid_constant__ TcParams P) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    const TcArgs& a = P.a;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    unsigned char* smem = (unsigned char*)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smemA = saddr(smem);
    const uint32_t smemB = smemA + TC_STAGES * TC_A_BYTES;
    TcCtl* ctl = (TcCtl*)(smem + TC_STAGES * (TC_A_BYTES + TC_B_BYTES));

    if (tid == 0) {
        for (int i = 0; i < TC_STAGES; ++i) {
            mbar_init(saddr(&ctl->full[i]), 1);
            mbar_init(saddr(&ctl->empty[i]), 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(saddr(&ctl->tfull[i]), 1);
            mbar_init(saddr(&ctl->tempty[i]), TC_EPI_THREADS);
        }
        ctl->abort_flag = 0;
        ctl->issued = 0;
        ctl->wait_cycles = a.wait_cycles;
        ctl->last_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_all();
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(saddr(&ctl->tmem_base)),
                     "r"((uint32_t)TC_TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    // the split of the attention units (the same for every step) and this CTA's ring items per step
    const TcAttInfo ai = tc_att_info<GQ>(a, cta, G);
    if (warp == 0) {
        if (lane == 0) tc_producer_w<DH, GQ>(P, ctl, smemA, cta, G, ai);
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) tc_mma_issuer(P, ctl, smemA, smemB, cta, G, ai.total);
        __syncwarp();
    } else if (warp == 2) {
        if (lane == 0) tc_producer_x(P, ctl, smemB, cta, G, ai.total);
        __syncwarp();
    } else if (warp >= 4) {
        // warps 4..7: the embedding gather at the start of a step, the epilogue of every GEMM phase and the attention
        // between the QKV and O phases
        // (warp 3 has no role: the epilogue warps must be warps 4..7, since a warp reads the 32 lanes of tensor memory
        // that its number modulo 4 selects)
        const int atid = tid - 32 * TC_ATT_FIRST;
        const bool is_epi = true;
        const int w4 = warp - 4;
        unsigned seg_cnt = 0;
        AttnWArgs aw;
        aw.qkv = a.qkv; aw.ld = a.qw + 2 * a.kvw; aw.Kc = (bf16*)a.Kc; aw.Vc = (bf16*)a.Vc; aw.slots = a.slots;
        aw.pos0 = a.pos0; aw.step = 0; aw.rope_tab = a.rope_tab; aw.Hq = a.Hq; aw.Hkv = a.Hkv; aw.max_len = a.max_len;
        aw.B = a.B; aw.scale = a.scale; aw.part_acc = a.part_acc; aw.part_ml = a.part_ml; aw.nslot = a.attn_nslot;
        aw.counters = a.counters; aw.attn = a.attn; aw.attn_h = a.attn_h; aw.lo_rows = a.lo;
        // ring items of this CTA per step, and those before the attention items of step 0
        unsigned items_step = ai.total, items_before = 0;
        for (int p = 0; p < PH_COUNT; ++p) {
            const PhaseShape sh = phase_shape(a, p);
            const unsigned cnt = (unsigned)(range_lo(sh.W, cta + 1, G) - range_lo(sh.W, cta, G));
            items_step += cnt;
            if (p < PH_O) items_before += cnt;
        }
        TcAttRing ring;
        ring.ctl = ctl; ring.error_flag = a.error_flag; ring.smemA = smemA; ring.w = warp - TC_ATT_FIRST;
#pragma unroll
        for (int w = 0; w < TC_ATT_WARPS; ++w) ring.n[w] = ai.n[w];
        for (int s = 0; s < a.k; ++s) {
            if (is_epi) {
                tc_gather(P, ctl, s, cta, G, atid);
                tc_epilogue_phase<SMP>(P, ctl, s, PH_FC, seg_cnt, cta, G, w4, lane);
                tc_epilogue_phase<SMP>(P, ctl, s, PH_QKV, seg_cnt, cta, G, w4, lane);
            }
            // ---- attention: needs every CTA's QKV rows
            if (seq_on(a, TC_SEQ_ATTN)) {
            if (atid == 0)
                wait_grid(a.bar_counter, a.bar_base + (u64)G * (u64)(s * TC_BARS_PER_STEP + TC_SEQ_ATTN), ctl, a.error_flag, 7);
            if (atid == 0) phase_stamp(a, s, 20, cta, G);
            named_sync(TC_BAR_ATT, TC_ATT_WARPS * 32);
            if (!poisoned(ctl)) {
                aw.step = s;
                aw.rope_tab = a.rope_tab + (long long)(s & 1) * 16 * (DH / 2);
                ring.base = items_before + (unsigned)s * items_step;
                if constexpr (AttSel<GQ>::mma) attn_mma_phase<DH, GQ>(aw, ai.job[warp - TC_ATT_FIRST], lane, ring);
                else attn_warp_phase<DH, GQ>(aw, ai.pl, (warp - TC_ATT_FIRST) * G + cta, lane, ring);
            }
            named_sync(TC_BAR_ATT, TC_ATT_WARPS * 32);
            if (atid == 0) {
                phase_stamp(a, s, TC_SEQ_ATTN, cta, G);
                red_release_add_u64(a.bar_counter, 1ull);
            }
            }
            if (is_epi) {
                tc_epilogue_phase<SMP>(P, ctl, s, PH_O, seg_cnt, cta, G, w4, lane);
                tc_epilogue_phase<SMP>(P, ctl, s, PH_GU, seg_cnt, cta, G, w4, lane);
                tc_epilogue_phase<SMP>(P, ctl, s, PH_DOWN, seg_cnt, cta, G, w4, lane);
                tc_epilogue_phase<SMP>(P, ctl, s, PH_LM, seg_cnt, cta, G, w4, lane);
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(ctl->tmem_base), "r"((uint32_t)TC_TMEM_COLS)
                     : "memory");
    }
}

// ------------------------------------------------------------------------------------------ set-up kernel
__global__ void tc_setup_kernel(SlotList sl, int k, int d, int lo, int* d_slots, int* d_pos0, int* kv_len,
                                const float* pend_feat, const int* pend_id, float* feat, bf16* feat_h, int* cur_id,
                                u64* keys, int key_stride, const bf16* embed, int vocab, bf16* xe_h, int* id_flag) {
    const int b = blockIdx.x;
    if (b >= sl.n) {
        // Rows of the embedding operand beyond the batch: the tiled copy always brings all rows, and the accumulator
        // columns of the remainder rows are added to those of the batch rows (an embedding row is exact in bf16, so
        // its remainder is zero).  An earlier, larger batch may have left rows here.
        for (int i = threadIdx.x; i < (d >> 3); i += blockDim.x)
            ((uint4*)(xe_h + (long long)b * d))[i] = make_uint4(0u, 0u, 0u, 0u);
        return;
    }
    const int slot = sl.slot[b];
    if (threadIdx.x == 0) {
        d_slots[b] = slot;
        const int rows = kv_len[slot];
        d_pos0[b] = rows;
        kv_len[slot] = rows + k;            // every draft step appends one K/V row
        cur_id[b] = pend_id[slot];
    }
    if (threadIdx.x < k) keys[(long long)b * key_stride + threadIdx.x] = 0ull;
    for (int i = threadIdx.x; i < d; i += blockDim.x) {
        const float v = pend_feat[(long long)slot * d + i];
        feat[(long long)b * d + i] = v;
        const bf16 hi = __float2bfloat16_rn(v);
        feat_h[(long long)b * d + i] = hi;
        if (lo) feat_h[(long long)(b + lo) * d + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
    }
    // embedding row of the pending token: the fusion FC's embedding operand of step 0
    const int id = checked_token(pend_id[slot], vocab, id_flag);
    for (int i = threadIdx.x; i < (d >> 3); i += blockDim.x)
        ((uint4*)(xe_h + (long long)b * d))[i] = ((const uint4*)(embed + (long long)id * d))[i];
}
cudaError_t launch_tc_setup(const SlotList& sl, int k, int d, int lo, int* d_slots, int* d_pos0, int* kv_len,
                            const float* pend_feat, const int* pend_id, float* feat, bf16* feat_h, int* cur_id,
                            u64* keys, int key_stride, const bf16* embed, int vocab, bf16* xe_h, int* id_flag,
                            cudaStream_t st) {
    tc_setup_kernel<<<TC_OP_ROWS, 256, 0, st>>>(sl, k, d, lo, d_slots, d_pos0, kv_len, pend_feat, pend_id, feat, feat_h,
                                                cur_id, keys, key_stride, embed, vocab, xe_h, id_flag);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 row-major [rows][cols] matrix, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside
static cudaError_t encode_map(unsigned char* out, const void* base, long long rows, long long cols, int box_rows,
                              CUtensorMapL2promotion promo) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return cudaErrorNotSupported;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {TC_BK, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides,
                          box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

bool tc_supported(int d, int dh, int Hq, int Hkv, int F) {
    return d % TC_BK == 0 && (dh == 64 || dh == 128) && Hkv > 0 && Hq % Hkv == 0 && F % 8 == 0;
}

int tc_max_tiles(const ChainPhase* ph) {
    int m = 0;
    for (int p = 0; p < PH_COUNT; ++p) {
        const int t = (ph[p].N + TC_TM - 1) / TC_TM;
        if (t > m) m = t;
    }
    return m;
}

int tc_barriers_per_step() { return TC_BARS_PER_STEP; }

// Row offset of the rounding remainders in the operand buffers for a batch of B (0: none are kept).
int tc_lo_offset(int B) {
#if TC_TN == 32
    (void)B;
    return 16;
#else
    return B <= 8 ? B : 0;
#endif
}

cudaError_t tc_build_maps(TcMaps* maps, const ChainPhase* ph, int d, int qw, int F,
                          const bf16* feat_h, const bf16* xq_h, const bf16* attn_h, const bf16* xm_h,
                          const bf16* act_h, const bf16* xe_h, const void* Kc, const void* Vc, long long cache_rows, int dh) {
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    cudaError_t e;
    for (int p = 0; p < PH_COUNT; ++p) {
        e = encode_map(maps->m[TCM_W + p], ph[p].W, ph[p].N, ph[p].K, TC_TM, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
        if (e != cudaSuccess) return e;
    }
    const struct { int idx; const bf16* base; int cols; } ops[5] = {
        {TCM_X_FEAT, feat_h, d}, {TCM_X_XQ, xq_h, d}, {TCM_X_ATTN, attn_h, qw}, {TCM_X_XM, xm_h, d}, {TCM_X_ACT, act_h, F}};
    for (int i = 0; i < 5; ++i) {
        e = encode_map(maps->m[ops[i].idx], ops[i].base, TC_OP_ROWS, ops[i].cols, TC_TN, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
        if (e != cudaSuccess) return e;
    }
    e = encode_map(maps->m[TCM_X_EMB], xe_h, TC_OP_ROWS, d, TC_TN, CU_TENSOR_MAP_L2_PROMOTION_L2_128B);
    if (e != cudaSuccess) return e;
    // the caches as matrices of [slot x KV head x position] rows: boxes of 32 rows x 64 elements
    e = encode_map(maps->m[TCM_K], Kc, cache_rows, dh, 32, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
    if (e != cudaSuccess) return e;
    return encode_map(maps->m[TCM_V], Vc, cache_rows, dh, 32, CU_TENSOR_MAP_L2_PROMOTION_L2_256B);
}

template <int DH, int GQ, bool SMP>
static cudaError_t tc_launch_t(const TcParams& P, int grid, cudaStream_t st) {
    // the shared-memory opt-in is a per-device attribute of the function: remember it per device ordinal
    static bool attr_set[HIVIS_MAX_DEVICES] = {false};
    const size_t smem = 1024 + (size_t)TC_STAGES * (TC_A_BYTES + TC_B_BYTES) + ((sizeof(TcCtl) + 127) & ~(size_t)127);
    if (smem > 227 * 1024) return cudaErrorInvalidValue;
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= HIVIS_MAX_DEVICES || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(tc_chain_kernel<DH, GQ, SMP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < HIVIS_MAX_DEVICES) attr_set[dev] = true;
    }
    void* params[] = {(void*)&P};
    return cudaLaunchCooperativeKernel((const void*)tc_chain_kernel<DH, GQ, SMP>, dim3(grid), dim3(TC_THREADS), params, smem, st);
}

cudaError_t launch_tc_chain(const TcMaps& maps, const TcArgs& a, int grid, cudaStream_t st) {
    TcParams P;
    P.maps = maps;
    P.a = a;
    const int G = a.Hq / a.Hkv;
    const int gq = (G % 7 == 0) ? 7 : 1;
    if (a.gumbel_u) {
        if (a.dh == 128) return gq == 7 ? tc_launch_t<128, 7, true>(P, grid, st) : tc_launch_t<128, 1, true>(P, grid, st);
        return gq == 7 ? tc_launch_t<64, 7, true>(P, grid, st) : tc_launch_t<64, 1, true>(P, grid, st);
    }
    if (a.dh == 128) return gq == 7 ? tc_launch_t<128, 7, false>(P, grid, st) : tc_launch_t<128, 1, false>(P, grid, st);
    return gq == 7 ? tc_launch_t<64, 7, false>(P, grid, st) : tc_launch_t<64, 1, false>(P, grid, st);
}
