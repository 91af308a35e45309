// Persistent draft-chain kernel for one sequence: all k chained draft steps in ONE cooperative launch.
//
// One CTA per SM, 16 warps.  Every weight matrix of the step (fusion FC, QKV, O, gate/up, down, LM
// head) is split by rows across the CTAs; inside a CTA the rows are cut into chunks of at most 4 KB of
// contiguous weights ("units") which the warps take round-robin.  Each warp owns a private ring of
// shared-memory stages and keeps it full with bulk-async copies (cp.async.bulk + mbarrier
// complete_tx): after it has consumed a stage it refills that stage itself with the unit that lies
// STAGES units ahead in ITS OWN unit sequence, and that sequence runs on across phase and step
// boundaries.  Weights do not depend on activations, so while a CTA finishes a phase, waits at the grid
// barrier and stages the next activation vector, the first units of the next phase are already
// landing in its rings: HBM keeps streaming through every dependency of the chain.
//
// Phases of a step (grid barrier after each):
//   FC (+rho) -> QKV (RMSNorm in the input stage) -> attention (RoPE, KV append, split-KV, arrival-
//   counter merge) -> O (+u) -> gate/up (RMSNorm in, SiLU*up out) -> down (+y) -> LM head + argmax.
// Partial dot products of a row's chunks go to shared-memory slots and are added in chunk order, the
// argmax is an integer max over packed (value, index) keys: results do not depend on timing.
//
// Every wait is bounded (grid barrier, mbarrier): when a bound is hit the kernel raises an error
// flag, waits (bounded) for its own copies in flight and returns.
#include "attn_body.cuh"

#ifndef CHAIN_WARPS
#define CHAIN_WARPS 16
#endif
#define CHAIN_THREADS (CHAIN_WARPS * 32)
#ifndef CHAIN_STAGES
#define CHAIN_STAGES 2
#endif
#ifndef CHAIN_CHUNK_BYTES
#define CHAIN_CHUNK_BYTES 4096
#endif

// ------------------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ u64 make_evict_first_policy() {
    u64 pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// contiguous global -> shared copy by the bulk-copy engine; completion is counted in bytes on `bar`
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, u64 pol) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
        ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol)
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ u64 ld_acquire_u64(const u64* p) {
    u64 v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add_u64(u64* p, u64 v) {
    asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ int ld_relaxed_int(const int* p) {
    int v;
    asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

struct ChainMisc {
    float red[CHAIN_WARPS];
    u64 kred[CHAIN_WARPS];
    int abort_flag;
    int r0[PH_COUNT];          // first row of this CTA in each phase
    int units[PH_COUNT];       // number of units of this CTA in each phase
    int cpr[PH_COUNT];         // chunks per row
};

// Grid-wide barrier on a monotonically increasing counter.  false = gave up (error flag raised).
__device__ __forceinline__ bool grid_barrier(const ChainArgs& a, ChainMisc* misc, u64 target) {
    __syncthreads();
    if (threadIdx.x == 0) {
        red_release_add_u64(a.bar_counter, 1ull);
        const long long t0 = clock64();
        unsigned it = 0;
        bool ok = true;
        while (ld_acquire_u64(a.bar_counter) < target) {
            if ((++it & 255u) == 0u && (ld_relaxed_int(a.error_flag) != 0 || clock64() - t0 > a.wait_cycles)) {
                ok = false;
                break;
            }
        }
        if (!ok) {
            atomicExch(a.error_flag, 1);
            misc->abort_flag = 1;
        }
    }
    __syncthreads();
    return misc->abort_flag == 0;
}

template <typename WT>
__device__ __forceinline__ int x_index(int k, int K) {
    if (sizeof(WT) == 2) return ((k >> 3) << 2) + (k & 3) + ((k >> 2) & 1) * (K >> 1);
    return k;
}

__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < CHAIN_WARPS; ++w) tot += red[w];
    return tot;
}

// dot product of one staged chunk with the matching slice of x
template <typename WT>
__device__ __forceinline__ float dot_chunk(const uint4* wsm, const float* xs, int K, int k0, int nvec, int lane) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (sizeof(WT) == 2) {
        const float4* xlo = (const float4*)xs + (k0 >> 3);
        const float4* xhi = (const float4*)(xs + (K >> 1)) + (k0 >> 3);
#pragma unroll 4
        for (int j = lane; j < nvec; j += 32) {
            const uint4 w = wsm[j];
            const float4 xa = xlo[j], xb = xhi[j];
            a0 = fmaf(bf16_lo(w.x), xa.x, a0); a1 = fmaf(bf16_hi(w.x), xa.y, a1);
            a2 = fmaf(bf16_lo(w.y), xa.z, a2); a3 = fmaf(bf16_hi(w.y), xa.w, a3);
            a0 = fmaf(bf16_lo(w.z), xb.x, a0); a1 = fmaf(bf16_hi(w.z), xb.y, a1);
            a2 = fmaf(bf16_lo(w.w), xb.z, a2); a3 = fmaf(bf16_hi(w.w), xb.w, a3);
        }
    } else {
        const float4* x4 = (const float4*)xs + (k0 >> 2);
#pragma unroll 4
        for (int j = lane; j < nvec; j += 32) {
            const uint4 w = wsm[j];
            const float4 xa = x4[j];
            a0 = fmaf(__uint_as_float(w.x), xa.x, a0); a1 = fmaf(__uint_as_float(w.y), xa.y, a1);
            a2 = fmaf(__uint_as_float(w.z), xa.z, a2); a3 = fmaf(__uint_as_float(w.w), xa.w, a3);
        }
    }
    float acc = (a0 + a1) + (a2 + a3);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    return acc;
}

template <typename WT, int DH>
__global__ void __launch_bounds__(CHAIN_THREADS, 1) draft_chain_kernel(const ChainArgs a) {
    extern __shared__ __align__(128) unsigned char smem[];
    constexpr int ES = (int)sizeof(WT);
    constexpr int CE = CHAIN_CHUNK_BYTES / ES;              // elements per full chunk
    float* xs = (float*)(smem + a.off_x);
    float* part = (float*)(smem + a.off_part);
    u64* bars = (u64*)(smem + a.off_bar);
    ChainMisc* misc = (ChainMisc*)(smem + a.off_misc);
    AttnSmem<CHAIN_WARPS, 1, DH>* asm_ = (AttnSmem<CHAIN_WARPS, 1, DH>*)(smem + a.off_x);   // x is idle during attention

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int cta = blockIdx.x, G = gridDim.x;
    const int d = a.d;

    if (tid == 0) {
        misc->abort_flag = 0;
        for (int p = 0; p < PH_COUNT; ++p) {
            const long long N = a.ph[p].N;
            long long r0, r1;
            if (p == PH_GU) {                                // keep (gate_i, up_i) row pairs together
                r0 = 2 * ((N / 2) * cta / G);
                r1 = 2 * ((N / 2) * (cta + 1) / G);
            } else {
                r0 = N * cta / G;
                r1 = N * (cta + 1) / G;
            }
            const int cpr = (a.ph[p].K * ES + CHAIN_CHUNK_BYTES - 1) / CHAIN_CHUNK_BYTES;
            misc->r0[p] = (int)r0;
            misc->cpr[p] = cpr;
            misc->units[p] = (int)(r1 - r0) * cpr;
        }
        for (int i = 0; i < CHAIN_WARPS * CHAIN_STAGES; ++i) mbar_init(smem_addr(bars + i), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    const int slot = a.slot;
    const int pos0 = a.kv_len[slot];
    if (cta == 0 && tid < a.k) a.keys[tid] = 0ull;       // consumed after several grid barriers

    // ---------------------------------------------------------------- per-warp weight stream
    const u64 pol = make_evict_first_policy();
    const uint32_t ring0 = smem_addr(smem) + warp * (CHAIN_STAGES * CHAIN_CHUNK_BYTES);
    const uint32_t bar0 = smem_addr(bars + warp * CHAIN_STAGES);
    unsigned fi = 0, ci = 0;                                // units fetched / consumed by this warp
    int f_step = 0, f_ph = 0, f_u = warp;                   // fetch cursor
    bool f_live = true;
    auto f_normalise = [&]() {                              // move the cursor to the next existing unit
        while (f_live && f_u >= misc->units[f_ph]) {
            f_u = warp;
            if (++f_ph == PH_COUNT) {
                f_ph = 0;
                if (++f_step == a.k) f_live = false;
            }
        }
    };
    auto fetch_next = [&]() {                               // lane 0 issues; every lane tracks the cursor
        if (!f_live) return;
        const ChainPhase& P = a.ph[f_ph];
        const int cpr = misc->cpr[f_ph];
        const int row = misc->r0[f_ph] + f_u / cpr;
        const int ch = f_u % cpr;
        const int k0 = ch * CE;
        const int len = min(CE, P.K - k0);
        if (lane == 0) {
            const unsigned st = fi % CHAIN_STAGES;
            const uint32_t bar = bar0 + st * 8;
            const char* src = (const char*)P.W + ((long long)row * P.K + k0) * ES;
            mbar_expect_tx(bar, (uint32_t)(len * ES));
            bulk_g2s(ring0 + st * CHAIN_CHUNK_BYTES, src, (uint32_t)(len * ES), bar, pol);
        }
        ++fi;
        f_u += CHAIN_WARPS;
        f_normalise();
    };
    f_normalise();
    for (int i = 0; i < CHAIN_STAGES; ++i) fetch_next();

    // consume this warp's units of phase p: partial dot products into part[u]
    auto consume_phase = [&](int p) -> bool {
        const int K = a.ph[p].K, cpr = misc->cpr[p], U = misc->units[p];
        for (int u = warp; u < U; u += CHAIN_WARPS) {
            const unsigned st = ci % CHAIN_STAGES;
            const uint32_t parity = (ci / CHAIN_STAGES) & 1u;
            const uint32_t bar = bar0 + st * 8;
            if (!mbar_try_wait(bar, parity)) {
                const long long t0 = clock64();
                while (!mbar_try_wait(bar, parity)) {
                    if (clock64() - t0 > a.wait_cycles) {
                        atomicExch(a.error_flag, 2);
                        misc->abort_flag = 1;
                        return false;
                    }
                }
            }
            const int ch = u % cpr;
            const int k0 = ch * CE;
            const int len = min(CE, K - k0);
            const uint4* wsm = (const uint4*)(smem + (size_t)(warp * CHAIN_STAGES + st) * CHAIN_CHUNK_BYTES);
            const float acc = dot_chunk<WT>(wsm, xs, K, k0, (len * ES) >> 4, lane);
            if (lane == 0) part[u] = acc;
            ++ci;
            __syncwarp();
            fence_proxy_async();                            // our reads of the stage precede its refill
            fetch_next();
        }
        return true;
    };
    auto row_sum = [&](int p, int rl) {                     // add a row's chunk partials in chunk order
        const int cpr = misc->cpr[p];
        float v = 0.f;
        for (int c = 0; c < cpr; ++c) v += part[rl * cpr + c];
        return v;
    };

    u64 bar_target = a.bar_base;
    bool alive = true;
    auto barrier = [&]() {
        bar_target += (u64)G;
        alive = grid_barrier(a, misc, bar_target);
        return alive;
    };

    AttnArgs aa;
    aa.qkv = a.qkv; aa.ld = a.qw + 2 * a.kvw; aa.Kc = a.Kc; aa.Vc = a.Vc; aa.slots = nullptr; aa.pos0 = nullptr;
    aa.step = 0; aa.inv_freq = a.inv_freq; aa.Hq = a.Hq; aa.Hkv = a.Hkv; aa.dh = a.dh; aa.max_len = a.max_len;
    aa.B = 1; aa.scale = a.scale; aa.chunk = a.attn_chunk; aa.nsplit = a.attn_nsplit; aa.part_acc = a.part_acc;
    aa.part_ml = a.part_ml; aa.counters = a.counters; aa.attn = a.attn; aa.attn_h = nullptr; aa.lo_rows = 0;

    for (int s = 0; s < a.k && alive; ++s) {
        // ============================================================ fusion FC + residual
        {
            const int K = 2 * d;
            int tok;
            if (s == 0) tok = a.pend_id[slot];
            else if (a.forced) tok = a.forced[s - 1];
            else tok = key_index(__ldcg(a.keys + (s - 1)));
            tok = checked_token(tok, a.V, a.id_flag);
            const float* f = s == 0 ? a.pend_feat + (long long)slot * d : a.feat;
            const long long e0 = (long long)tok * d;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS)
                xs[x_index<WT>(kk, K)] = kk < d ? __ldcg(f + kk) : load_as_float<WT>(a.embed, e0 + (kk - d));
            __syncthreads();
            if (!consume_phase(PH_FC)) {}
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_FC], rows = misc->units[PH_FC] / misc->cpr[PH_FC];
            const float* rho = a.rho ? a.rho + (long long)(s < a.n_resid - 1 ? s : a.n_resid - 1) * d : nullptr;
            for (int rl = tid; rl < rows; rl += CHAIN_THREADS)
                a.u[r0 + rl] = row_sum(PH_FC, rl) + (rho ? rho[r0 + rl] : 0.f);
            if (!barrier()) break;
        }
        // ============================================================ RMSNorm + QKV
        {
            const int K = d;
            float ss = 0.f;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) {
                const float v = __ldcg(a.u + kk);
                ss += v * v;
                xs[x_index<WT>(kk, K)] = v;
            }
            const float inv = rsqrtf(block_sum(ss, misc->red) / (float)K + a.eps);
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) {
                const int i = x_index<WT>(kk, K);
                xs[i] = xs[i] * load_as_float<WT>(a.norm1, kk) * inv;
            }
            __syncthreads();
            consume_phase(PH_QKV);
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_QKV], rows = misc->units[PH_QKV] / misc->cpr[PH_QKV];
            for (int rl = tid; rl < rows; rl += CHAIN_THREADS)
                a.qkv[r0 + rl] = row_sum(PH_QKV, rl) + (a.bqkv ? load_as_float<WT>(a.bqkv, r0 + rl) : 0.f);
            if (!barrier()) break;
        }
        // ============================================================ attention over the text-only cache
        {
            const int nunits = a.Hq * a.attn_nsplit;
            for (int unit = cta; unit < nunits; unit += G)
                attn_unit<WT, DH, 1, CHAIN_WARPS>(aa, unit % a.attn_nsplit, unit / a.attn_nsplit, 0, pos0 + s, slot, *asm_);
            if (!barrier()) break;
        }
        // ============================================================ O projection + residual
        {
            const int K = a.qw;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) xs[x_index<WT>(kk, K)] = __ldcg(a.attn + kk);
            __syncthreads();
            consume_phase(PH_O);
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_O], rows = misc->units[PH_O] / misc->cpr[PH_O];
            for (int rl = tid; rl < rows; rl += CHAIN_THREADS)
                a.y[r0 + rl] = __ldcg(a.u + r0 + rl) + row_sum(PH_O, rl);
            if (!barrier()) break;
        }
        // ============================================================ RMSNorm + gate/up + SiLU*up
        {
            const int K = d;
            float ss = 0.f;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) {
                const float v = __ldcg(a.y + kk);
                ss += v * v;
                xs[x_index<WT>(kk, K)] = v;
            }
            const float inv = rsqrtf(block_sum(ss, misc->red) / (float)K + a.eps);
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) {
                const int i = x_index<WT>(kk, K);
                xs[i] = xs[i] * load_as_float<WT>(a.norm2, kk) * inv;
            }
            __syncthreads();
            consume_phase(PH_GU);
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_GU], rows = misc->units[PH_GU] / misc->cpr[PH_GU];
            for (int pl = tid; pl < rows / 2; pl += CHAIN_THREADS) {
                const float gate = row_sum(PH_GU, 2 * pl), up = row_sum(PH_GU, 2 * pl + 1);
                a.act[r0 / 2 + pl] = gate / (1.f + expf(-gate)) * up;
            }
            if (!barrier()) break;
        }
        // ============================================================ down projection + residual
        {
            const int K = a.F;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) xs[x_index<WT>(kk, K)] = __ldcg(a.act + kk);
            __syncthreads();
            consume_phase(PH_DOWN);
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_DOWN], rows = misc->units[PH_DOWN] / misc->cpr[PH_DOWN];
            for (int rl = tid; rl < rows; rl += CHAIN_THREADS)
                a.feat[r0 + rl] = __ldcg(a.y + r0 + rl) + row_sum(PH_DOWN, rl);
            if (!barrier()) break;
        }
        // ============================================================ LM head + argmax
        {
            const int K = d;
            for (int kk = tid; kk < K; kk += CHAIN_THREADS) xs[x_index<WT>(kk, K)] = __ldcg(a.feat + kk);
            __syncthreads();
            consume_phase(PH_LM);
            __syncthreads();
            if (misc->abort_flag) break;
            const int r0 = misc->r0[PH_LM], rows = misc->units[PH_LM] / misc->cpr[PH_LM];
            u64 best = 0;
            for (int rl = tid; rl < rows; rl += CHAIN_THREADS) {
                const float v = row_sum(PH_LM, rl);
                if (a.logits_out) a.logits_out[(long long)s * a.V + r0 + rl] = v;
                const u64 key = a.gumbel_u ? pack_key(gumbel_perturbed(v, a.inv_t, __ldg(a.gumbel_u + (long long)s * a.V + r0 + rl)), r0 + rl)
                                           : pack_key(v, r0 + rl);
                best = key > best ? key : best;
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
                best = other > best ? other : best;
            }
            if (lane == 0) misc->kred[warp] = best;
            __syncthreads();
            if (tid == 0) {
                u64 m = misc->kred[0];
#pragma unroll
                for (int w = 1; w < CHAIN_WARPS; ++w) m = misc->kred[w] > m ? misc->kred[w] : m;
                if (m) atomicMax(a.keys + s, m);
            }
            if (!barrier()) break;
        }
    }
    if (alive && misc->abort_flag == 0) {
        if (cta == 0) {
            if (tid < a.k) a.out_ids[tid] = key_index(__ldcg(a.keys + tid));
            if (tid == 0) a.kv_len[slot] = pos0 + a.k;
        }
        return;                                             // every fetched unit has been consumed
    }
    // gave up: wait (bounded) for this warp's copies that are still in flight, then leave
    for (; ci < fi; ++ci) {
        const uint32_t bar = bar0 + (ci % CHAIN_STAGES) * 8;
        const uint32_t parity = (ci / CHAIN_STAGES) & 1u;
        const long long t0 = clock64();
        while (!mbar_try_wait(bar, parity))
            if (clock64() - t0 > a.wait_cycles) break;
    }
}

// ------------------------------------------------------------------------------------------ host side
struct ChainPlan {
    int off_x, off_part, off_bar, off_misc;
    size_t smem_bytes;
};

static ChainPlan chain_plan(const ChainArgs& a, int es, int dh, int grid) {
    ChainPlan p;
    int kmax = 0;
    long long slots = 0;
    for (int i = 0; i < PH_COUNT; ++i) {
        if (a.ph[i].K > kmax) kmax = a.ph[i].K;
        const long long rows = (a.ph[i].N + grid - 1) / grid + 2;
        const long long cpr = ((long long)a.ph[i].K * es + CHAIN_CHUNK_BYTES - 1) / CHAIN_CHUNK_BYTES;
        if (rows * cpr > slots) slots = rows * cpr;
    }
    size_t x_bytes = (size_t)kmax * 4;
    const size_t attn_bytes = dh == 128 ? sizeof(AttnSmem<CHAIN_WARPS, 1, 128>) : sizeof(AttnSmem<CHAIN_WARPS, 1, 64>);
    if (attn_bytes > x_bytes) x_bytes = attn_bytes;
    size_t off = (size_t)CHAIN_WARPS * CHAIN_STAGES * CHAIN_CHUNK_BYTES;
    p.off_x = (int)off;
    off += (x_bytes + 127) & ~(size_t)127;
    p.off_part = (int)off;
    off += ((size_t)slots * 4 + 127) & ~(size_t)127;
    p.off_bar = (int)off;
    off += CHAIN_WARPS * CHAIN_STAGES * 8;
    off = (off + 15) & ~(size_t)15;
    p.off_misc = (int)off;
    off += sizeof(ChainMisc);
    p.smem_bytes = off;
    return p;
}

int chain_barriers_per_step() { return 7; }

template <typename WT, int DH>
static cudaError_t chain_launch_t(ChainArgs& a, int grid, size_t smem, cudaStream_t st) {
    // the shared-memory opt-in is a per-device attribute of the function: remember it per device ordinal
    static size_t attr_smem[HIVIS_MAX_DEVICES] = {0};
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= HIVIS_MAX_DEVICES || smem > attr_smem[dev]) {
        cudaError_t e = cudaFuncSetAttribute(draft_chain_kernel<WT, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < HIVIS_MAX_DEVICES) attr_smem[dev] = smem;
    }
    void* params[] = {(void*)&a};
    return cudaLaunchCooperativeKernel((const void*)draft_chain_kernel<WT, DH>, dim3(grid), dim3(CHAIN_THREADS), params, smem, st);
}

// Shared-memory bytes the chain kernel needs for these dimensions (0 = does not fit).
size_t chain_smem_bytes(const ChainArgs& a, int dtype, int grid) {
    const ChainPlan p = chain_plan(a, dtype == HIVIS_BF16 ? 2 : 4, a.dh, grid);
    return p.smem_bytes <= 227 * 1024 ? p.smem_bytes : 0;
}

cudaError_t launch_draft_chain(ChainArgs& a, int dtype, int grid, cudaStream_t st) {
    const ChainPlan p = chain_plan(a, dtype == HIVIS_BF16 ? 2 : 4, a.dh, grid);
    if (p.smem_bytes > 227 * 1024) return cudaErrorInvalidValue;
    a.off_x = p.off_x; a.off_part = p.off_part; a.off_bar = p.off_bar; a.off_misc = p.off_misc;
    if (dtype == HIVIS_BF16)
        return a.dh == 128 ? chain_launch_t<bf16, 128>(a, grid, p.smem_bytes, st) : chain_launch_t<bf16, 64>(a, grid, p.smem_bytes, st);
    return a.dh == 128 ? chain_launch_t<float, 128>(a, grid, p.smem_bytes, st) : chain_launch_t<float, 64>(a, grid, p.smem_bytes, st);
}
