// Prefix build on the tensor cores (Algorithm 1, the prefix build; Eq. 1): for every packed (hidden state, token) pair
//     u = W_fc [h ; E[id]] + rho_0,   a = gamma_1 * u / rms(u),   K = RoPE(W_k a + b_k, position),   V = W_v a + b_v
// and K, V go to the pair's cache row.  Unlike a draft step this is a dense contraction - thousands of pairs share
// every weight tile - so it runs as two tcgen05 GEMMs with the weights as the M operand (128 rows) and 128 pairs
// as the N operand, both staged by TMA (128-byte swizzle) through a six-stage ring, accumulators in tensor memory:
//   GEMM 1 (fusion FC):  [d rows] x [2d] x pairs.  The k-blocks of the hidden half come from the caller's hidden
//                        states, those of the embedding half from a buffer of gathered embedding rows.  Output
//                        stage: + rho_0, per-pair partial sums of squares of the tile's rows, gamma_1 * u as bf16
//                        (pair-major, the operand of GEMM 2).  The RMSNorm scale is applied after GEMM 2.
//   GEMM 2 (K and V):    [2 * Hkv * dh rows] x [d] x pairs.  Output stage: scale by 1/rms, bias, rotate K at the
//                        pair's position, scatter 16-byte pieces to the cache rows; pending pairs (row -1) are skipped.
// One CTA computes one 128 x 128 output tile.  Warp 0 (one thread) issues the copies, warp 1 (one thread) the MMAs,
// warps 2-5 run the output stage: each thread reads its weight row of the accumulator, the tile is turned in
// shared memory (the ring is free by then) so that a thread then owns one PAIR and writes whole 16-byte pieces,
// and sums over rows run in a fixed order.  Every wait is bounded; a wait that runs out raises the error word.
#include <cuda.h>

#include "attn_body.cuh"

#define PF_THREADS 192
#define PF_STAGES 6
#define PF_BK 64
#define PF_TM 128
#define PF_TN 128
#define PF_A_BYTES (PF_TM * PF_BK * 2)
#define PF_B_BYTES (PF_TN * PF_BK * 2)
#define PF_LD (PF_TM + 1)              // row stride (floats) of the turned tile: [pair][weight row]
#define PF_IDESC ((1u << 4) | (1u << 7) | (1u << 10) | ((PF_TN >> 3) << 17) | ((PF_TM >> 4) << 24))

namespace {

struct PfCtl {
    u64 full[PF_STAGES], empty[PF_STAGES], tfull;
    uint32_t tmem_base;
    int abort_flag;
};

__device__ __forceinline__ uint32_t pf_saddr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void pf_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void pf_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool pf_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// bounded wait; false: gave up (error word raised, the CTA's other roles stop as well)
__device__ __forceinline__ bool pf_wait(uint32_t bar, uint32_t parity, PfCtl* ctl, long long limit, int* error_flag) {
    if (pf_try(bar, parity)) return true;
    const long long t0 = clock64();
    unsigned it = 0;
    while (!pf_try(bar, parity)) {
        if ((++it & 63u) == 0u) {
            if (*(volatile int*)&ctl->abort_flag) return false;
            if (clock64() - t0 > limit) {
                atomicCAS(error_flag, 0, 30);
                *(volatile int*)&ctl->abort_flag = 1;
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ void pf_tma_2d(uint32_t dst, const void* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
        "l"(map), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void pf_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void pf_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void pf_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void pf_mma(uint32_t d_tmem, u64 adesc, u64 bdesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"((uint32_t)PF_IDESC), "r"(accumulate)
        : "memory");
}
// K-major tile with 128-byte rows, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ u64 pf_smem_desc(uint32_t addr) {
    const uint32_t lo = ((addr >> 4) & 0x3FFFu) | (1u << 16);
    const uint32_t hi = (1024u >> 4) | (1u << 14) | (2u << 29);
    return ((u64)hi << 32) | lo;
}
__device__ __forceinline__ void pf_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,"
        "%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

struct PfParams {
    alignas(64) unsigned char map_w[128];      // weights [rows][K], box 64 x 128
    alignas(64) unsigned char map_x0[128];     // operand of k-blocks [0, kb_split): [pairs][.], box 64 x 128
    alignas(64) unsigned char map_x1[128];     // operand of k-blocks [kb_split, nkb)
    int rows, K, kb_split, n_pairs;
    long long wait_cycles;
    int* error_flag;
    // GEMM 1 output stage
    const float* rho;          // [rows] nullable
    const bf16* gamma;         // [rows]
    bf16* xq;                  // [pairs][rows]
    float* ssq;                // [row tiles][pair capacity]
    int pair_cap;
    // GEMM 2 output stage
    const float* ssq_in;       // [ssq_tiles][pair capacity]
    int ssq_tiles, d;
    float eps;
    const bf16* bias;          // [rows] nullable
    int kvw, Hkv, dh, max_len;
    const int *slot_of, *row_of;
    const float2* rope;        // [pairs][dh / 2] (cos, sin) at the pair's position
    bf16 *Kc, *Vc;
};

template <int EPI>   // 0: fusion FC, 1: K and V
__global__ void __launch_bounds__(PF_THREADS, 1) prefill_tc_kernel(const __grid_constant__ PfParams P) {
    extern __shared__ __align__(1024) unsigned char pf_smem_raw[];
    unsigned char* smem = (unsigned char*)(((uintptr_t)pf_smem_raw + 1023) & ~(uintptr_t)1023);
    const uint32_t smemA = pf_saddr(smem), smemB = smemA + PF_STAGES * PF_A_BYTES;
    PfCtl* ctl = (PfCtl*)(smem + PF_STAGES * (PF_A_BYTES + PF_B_BYTES));
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int row0 = blockIdx.x * PF_TM, pair0 = blockIdx.y * PF_TN;
    const int nkb = P.K / PF_BK;
    if (tid == 0) {
        for (int i = 0; i < PF_STAGES; ++i) {
            pf_mbar_init(pf_saddr(&ctl->full[i]), 1);
            pf_mbar_init(pf_saddr(&ctl->empty[i]), 1);
        }
        pf_mbar_init(pf_saddr(&ctl->tfull), 1);
        ctl->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(pf_saddr(&ctl->tmem_base)),
                     "r"((uint32_t)PF_TN)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pf_fence_before();
    __syncthreads();
    pf_fence_after();

    if (warp == 0) {
        if (lane == 0) {
            for (int kb = 0; kb < nkb; ++kb) {
                const int slot = kb % PF_STAGES, round = kb / PF_STAGES;
                if (round > 0 && !pf_wait(pf_saddr(&ctl->empty[slot]), (round - 1) & 1u, ctl, P.wait_cycles, P.error_flag)) break;
                const uint32_t bar = pf_saddr(&ctl->full[slot]);
                pf_expect_tx(bar, PF_A_BYTES + PF_B_BYTES);
                pf_tma_2d(smemA + slot * PF_A_BYTES, P.map_w, kb * PF_BK, row0, bar);
                if (kb < P.kb_split) pf_tma_2d(smemB + slot * PF_B_BYTES, P.map_x0, kb * PF_BK, pair0, bar);
                else pf_tma_2d(smemB + slot * PF_B_BYTES, P.map_x1, (kb - P.kb_split) * PF_BK, pair0, bar);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t tmem = ctl->tmem_base;
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int slot = kb % PF_STAGES, round = kb / PF_STAGES;
                ok = pf_wait(pf_saddr(&ctl->full[slot]), round & 1u, ctl, P.wait_cycles, P.error_flag);
                if (!ok) break;
                pf_fence_after();
                const u64 ad = pf_smem_desc(smemA + slot * PF_A_BYTES), bd = pf_smem_desc(smemB + slot * PF_B_BYTES);
#pragma unroll
                for (int kk = 0; kk < PF_BK / 16; ++kk) pf_mma(tmem, ad + (u64)(kk * 2), bd + (u64)(kk * 2), (kb > 0 || kk > 0) ? 1u : 0u);
                pf_commit(pf_saddr(&ctl->empty[slot]));
            }
            if (ok) pf_commit(pf_saddr(&ctl->tfull));
        }
        __syncwarp();
    } else {
        // ---- output stage: warps 2..5 read the tensor-memory lanes their number modulo 4 selects
        const int quarter = warp & 3, etid = tid - 64;                  // etid: 0..127
        const int r_loc = quarter * 32 + lane, row = row0 + r_loc;
        float* tile = (float*)smem;                                      // [PF_TN pairs][PF_LD]: the ring is free by now
        bool ok = true;
        if (lane == 0) ok = pf_wait(pf_saddr(&ctl->tfull), 0u, ctl, P.wait_cycles, P.error_flag);
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        pf_fence_after();
        if (ok) {
#pragma unroll 1
            for (int c0 = 0; c0 < PF_TN; c0 += 32) {
                float v[32];
                pf_ld32(ctl->tmem_base + ((uint32_t)(quarter * 32) << 16) + c0, v);
                if (EPI == 0) {
                    const float add = (P.rho && row < P.rows) ? P.rho[row] : 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) tile[(c0 + i) * PF_LD + r_loc] = v[i] + add;
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) tile[(c0 + i) * PF_LD + r_loc] = v[i];
                }
            }
        }
        pf_fence_before();
        asm volatile("bar.sync 1, 128;" ::: "memory");
        // ---- a thread now owns one pair of the tile
        const int pair = pair0 + etid;
        const float* mine = tile + etid * PF_LD;
        const int nrows = min(PF_TM, P.rows - row0);
        if (ok && !*(volatile int*)&ctl->abort_flag && pair < P.n_pairs) {
            if (EPI == 0) {
                float ss = 0.f;
                for (int r = 0; r < nrows; ++r) ss = fmaf(mine[r], mine[r], ss);
                P.ssq[(long long)blockIdx.x * P.pair_cap + pair] = ss;
                bf16* dst = P.xq + (long long)pair * P.rows + row0;
                for (int r = 0; r < nrows; r += 8) {
                    unsigned w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float x0 = __bfloat162float(P.gamma[row0 + r + 2 * e]) * mine[r + 2 * e];
                        const float x1 = __bfloat162float(P.gamma[row0 + r + 2 * e + 1]) * mine[r + 2 * e + 1];
                        w[e] = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(x0)) |
                               ((unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(x1)) << 16);
                    }
                    *(uint4*)(dst + r) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            } else {
                const int crow = P.row_of[pair];
                if (crow >= 0) {
                    float tot = 0.f;
                    for (int t = 0; t < P.ssq_tiles; ++t) tot += P.ssq_in[(long long)t * P.pair_cap + pair];
                    const float sc = rsqrtf(tot / (float)P.d + P.eps);
                    const int slot = P.slot_of[pair], half = P.dh >> 1;
                    for (int r = 0; r < nrows; r += 8) {
                        const int g = row0 + r;                               // row of the stacked [K ; V] projection
                        const bool isK = g < P.kvw;
                        const int gr = isK ? g : g - P.kvw, head = gr / P.dh, e0 = gr % P.dh;
                        unsigned w[4];
                        float x[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            float val = mine[r + e] * sc + (P.bias ? __bfloat162float(P.bias[g + e]) : 0.f);
                            if (isK) {
                                const int ee = e0 + e, f = ee % half;
                                const int pr = r + e + (ee < half ? half : -half);        // the partner row, in this tile
                                const float part = mine[pr] * sc + (P.bias ? __bfloat162float(P.bias[row0 + pr]) : 0.f);
                                const float2 t = __ldg(P.rope + (long long)pair * half + f);
                                val = ee < half ? val * t.x - part * t.y : val * t.x + part * t.y;
                            }
                            x[e] = val;
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = (unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(x[2 * e])) |
                                   ((unsigned)__bfloat16_as_ushort(__float2bfloat16_rn(x[2 * e + 1])) << 16);
                        bf16* base = isK ? P.Kc : P.Vc;
                        *(uint4*)(base + (((long long)slot * P.Hkv + head) * P.max_len + crow) * P.dh + e0) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }
    pf_fence_before();
    __syncthreads();
    if (warp == 1) {
        pf_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(ctl->tmem_base), "r"((uint32_t)PF_TN) : "memory");
    }
}

// embedding rows of the pairs' tokens, pair-major: the embedding half of GEMM 1's operand
__global__ void prefill_gather_kernel(const int32_t* ids, int n_pairs, int d, int vocab, const bf16* embed, bf16* xe, int* id_flag) {
    const int upr = d >> 3;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < (long long)n_pairs * upr; i += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(i / upr), off = (int)(i % upr);
        const int id = checked_token(ids[n], vocab, id_flag);
        ((uint4*)(xe + (long long)n * d))[off] = ld_stream((const uint4*)(embed + (long long)id * d) + off);
    }
}

// (cos, sin) of every pair's position, once per call: every K tile of GEMM 2 rotates with the same angles
__global__ void prefill_rope_kernel(const int* row_of, int n_pairs, int half, const double* inv_freq, float2* rope) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < (long long)n_pairs * half; i += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(i / half), f = (int)(i % half);
        const int pos = row_of[n];
        float cs = 1.f, sn = 0.f;
        if (pos >= 0) rope_cs(pos, inv_freq[f], cs, sn);
        rope[i] = make_float2(cs, sn);
    }
}

typedef CUresult (*PfEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
cudaError_t pf_encode(unsigned char* out, const void* base, long long rows, long long cols) {
    static PfEncodeFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return cudaErrorNotSupported;
        }
        fn = (PfEncodeFn)p;
    }
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {PF_BK, 128};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = fn((CUtensorMap*)out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <int EPI>
cudaError_t pf_launch(const PfParams& P, cudaStream_t st) {
    static bool attr_set[HIVIS_MAX_DEVICES] = {false};
    const size_t smem = 1024 + (size_t)PF_STAGES * (PF_A_BYTES + PF_B_BYTES) + 256;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= HIVIS_MAX_DEVICES || !attr_set[dev]) {
        e = cudaFuncSetAttribute(prefill_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < HIVIS_MAX_DEVICES) attr_set[dev] = true;
    }
    const dim3 grid((unsigned)((P.rows + PF_TM - 1) / PF_TM), (unsigned)((P.n_pairs + PF_TN - 1) / PF_TN));
    prefill_tc_kernel<EPI><<<grid, PF_THREADS, smem, st>>>(P);
    return cudaGetLastError();
}

}  // namespace

bool prefill_tc_supported(int d, int kvw) {
    static_assert(sizeof(CUtensorMap) == 128, "tensor map size");
    static_assert((size_t)PF_TN * PF_LD * 4 <= (size_t)PF_STAGES * (PF_A_BYTES + PF_B_BYTES), "the turned tile must fit in the ring");
    return d % PF_BK == 0 && (2 * kvw) % 8 == 0;
}

cudaError_t launch_prefill_tc(const PrefillTcArgs& a, cudaStream_t st) {
    const int d = a.d;
    prefill_gather_kernel<<<592, 256, 0, st>>>(a.ids, a.n_pairs, d, a.vocab, a.embed, a.xe, a.id_flag);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    prefill_rope_kernel<<<296, 256, 0, st>>>(a.row_of, a.n_pairs, a.dh / 2, a.inv_freq, a.rope);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    PfParams P;
    memset(&P, 0, sizeof(P));
    // ---- GEMM 1: u = W_fc [h ; E[id]] + rho_0
    if ((e = pf_encode(P.map_w, a.fc, d, 2 * d)) != cudaSuccess) return e;
    if ((e = pf_encode(P.map_x0, a.hidden, a.n_pairs, d)) != cudaSuccess) return e;
    if ((e = pf_encode(P.map_x1, a.xe, a.n_pairs, d)) != cudaSuccess) return e;
    P.rows = d; P.K = 2 * d; P.kb_split = d / PF_BK; P.n_pairs = a.n_pairs;
    P.wait_cycles = a.wait_cycles; P.error_flag = a.error_flag;
    P.rho = a.rho0; P.gamma = a.norm1; P.xq = a.xq; P.ssq = a.ssq; P.pair_cap = a.pair_cap;
    if ((e = pf_launch<0>(P, st)) != cudaSuccess) return e;
    // ---- GEMM 2: K, V
    PfParams Q;
    memset(&Q, 0, sizeof(Q));
    if ((e = pf_encode(Q.map_w, a.wkv, 2 * a.kvw, d)) != cudaSuccess) return e;
    if ((e = pf_encode(Q.map_x0, a.xq, a.n_pairs, d)) != cudaSuccess) return e;
    memcpy(Q.map_x1, Q.map_x0, 128);
    Q.rows = 2 * a.kvw; Q.K = d; Q.kb_split = d / PF_BK; Q.n_pairs = a.n_pairs;
    Q.wait_cycles = a.wait_cycles; Q.error_flag = a.error_flag;
    Q.ssq_in = a.ssq; Q.ssq_tiles = (d + PF_TM - 1) / PF_TM; Q.pair_cap = a.pair_cap; Q.d = d; Q.eps = a.eps;
    Q.bias = a.bkv; Q.kvw = a.kvw; Q.Hkv = a.Hkv; Q.dh = a.dh; Q.max_len = a.max_len;
    Q.slot_of = a.slot_of; Q.row_of = a.row_of; Q.rope = a.rope; Q.Kc = a.Kc; Q.Vc = a.Vc;
    return pf_launch<1>(Q, st);
}
