// Skinny linear layers of the drafter step: every projection of the decoder layer, the fusion
// FC and the LM head are  out[b][n] = sum_k W[n][k] x[b][k]  with at most a few batch rows, so
// each is one pass over W at HBM speed with the surrounding element-wise work fused in.
//
//   gemv_alu_kernel : one batch row per CTA column, fp32 FMAs, x staged in shared memory in fp32.
//                     Used for batch 1 and for fp32 weights.
//   gemm_mma_kernel : bf16 weights, 2..16 batch rows, mma.sync m16n8k16 with the weights as the
//                     M operand (16 weight rows) and the batch as N.  Weight fragments are loaded
//                     straight from global memory with 128-bit loads: a dot product does not care
//                     in which order k is visited, so lane (g,t) takes the 8 contiguous elements
//                     [32*blk + 8t, +8) of rows g and g+8 and feeds them to two MMAs, the batch
//                     operand using the same k order.
#include "hivis_internal.cuh"

// ------------------------------------------------------------------------------------------
// output stage for one batch row and one pair of adjacent weight rows (row is even)
// ------------------------------------------------------------------------------------------
template <typename WT, int EPI>
__device__ __forceinline__ void epilogue_pair(const LinArgs& a, int b, int row, float v0, float v1,
                                              bool has2, float scale, float& sq, u64& key) {
    const long long o = (long long)b * a.N + row;
    if (EPI == EPI_FUSE || EPI == EPI_OPROJ) {
        float r0, r1 = 0.f;
        if (EPI == EPI_FUSE) {
            r0 = v0 + (a.rho ? a.rho[row] : 0.f);
            if (has2) r1 = v1 + (a.rho ? a.rho[row + 1] : 0.f);
        } else {
            r0 = a.addend[o] + v0;
            if (has2) r1 = a.addend[o + 1] + v1;
        }
        a.out[o] = r0;
        if (has2) a.out[o + 1] = r1;
        if (a.out_h) {
            a.out_h[o] = __float2bfloat16_rn(load_as_float<WT>(a.gamma_out, row) * r0);
            if (has2) a.out_h[o + 1] = __float2bfloat16_rn(load_as_float<WT>(a.gamma_out, row + 1) * r1);
        }
        sq = r0 * r0 + r1 * r1;
    } else if (EPI == EPI_QKV) {
        a.out[o] = v0 * scale + (a.bias ? load_as_float<WT>(a.bias, row) : 0.f);
        if (has2) a.out[o + 1] = v1 * scale + (a.bias ? load_as_float<WT>(a.bias, row + 1) : 0.f);
    } else if (EPI == EPI_GATEUP) {   // row = gate_i, row + 1 = up_i, i = row / 2
        const float gate = v0 * scale, up = v1 * scale;
        const float act = gate / (1.f + expf(-gate)) * up;
        const long long oi = (long long)b * (a.N >> 1) + (row >> 1);
        if (a.out) a.out[oi] = act;
        if (a.out_h) a.out_h[oi] = __float2bfloat16_rn(act);
    } else if (EPI == EPI_DOWN) {
        const float r0 = a.addend[o] + v0;
        a.out[o] = r0;
        if (a.out_h) a.out_h[o] = __float2bfloat16_rn(r0);
        if (has2) {
            const float r1 = a.addend[o + 1] + v1;
            a.out[o + 1] = r1;
            if (a.out_h) a.out_h[o + 1] = __float2bfloat16_rn(r1);
        }
    } else {   // EPI_LM
        if (a.logits_out) {
            float* lo = a.logits_out + (long long)b * a.logits_ld + row;
            lo[0] = v0;
            if (has2) lo[1] = v1;
        }
        key = pack_key(v0, row);
        if (has2) {
            const u64 k1 = pack_key(v1, row + 1);
            key = k1 > key ? k1 : key;
        }
    }
}

__device__ __forceinline__ int fuse_token(const LinArgs& a, int b) {
    const int id = a.ids ? a.ids[(long long)b * a.id_stride] : key_index(a.keys[(long long)b * a.key_stride]);
    return checked_token(id, a.vocab, a.id_flag);
}

// ==========================================================================================
// gemv_alu
// ==========================================================================================
// Position of element k of x in shared memory.  For bf16 weights a 16-byte weight chunk holds 8
// elements; their x values are kept as two float4 (elements 0-3 and 4-7 of the chunk) in two
// separate arrays so that consecutive lanes read consecutive float4 (no bank conflicts).
template <typename WT>
__device__ __forceinline__ int xs_index(int k, int K) {
    if (sizeof(WT) == 2) return ((k >> 3) << 2) + (k & 3) + ((k >> 2) & 1) * (K >> 1);
    return k;
}

template <typename WT, int PRO>
__device__ __forceinline__ void load_x(const LinArgs& a, int b, float* xs, float* red) {
    const int K = a.K, tid = threadIdx.x;
    if (PRO == PRO_PLAIN) {
        const float* x = a.xin + (long long)b * K;
        for (int k = tid; k < K; k += 256) xs[xs_index<WT>(k, K)] = __ldcg(x + k);
    } else if (PRO == PRO_FUSE) {
        const int d = a.d;
        const float* f = a.feat + (long long)b * d;
        const long long e0 = (long long)fuse_token(a, b) * d;
        for (int k = tid; k < K; k += 256) {
            const float v = k < d ? __ldcg(f + k) : load_as_float<WT>(a.embed, e0 + (k - d));
            xs[xs_index<WT>(k, K)] = v;
        }
    } else {   // PRO_NORM
        const float* x = a.xin + (long long)b * K;
        float ss = 0.f;
        for (int k = tid; k < K; k += 256) {
            const float v = __ldcg(x + k);
            ss += v * v;
            xs[xs_index<WT>(k, K)] = v;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
        if ((tid & 31) == 0) red[tid >> 5] = ss;
        __syncthreads();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) tot += red[w];
        const float inv = rsqrtf(tot / (float)K + a.eps);
        for (int k = tid; k < K; k += 256) {
            const int i = xs_index<WT>(k, K);
            xs[i] = xs[i] * load_as_float<WT>(a.gamma, k) * inv;
        }
    }
    __syncthreads();
}

template <typename WT, int PRO, int EPI>
__global__ void __launch_bounds__(256) gemv_alu_kernel(const LinArgs a, int ppw) {
    extern __shared__ __align__(16) float xs[];
    __shared__ float red[8];
    __shared__ u64 kred[8];
    constexpr int U = 4;
    constexpr int VEC = 16 / (int)sizeof(WT);
    const int b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nch = a.K / VEC;
    const uint4 zero = make_uint4(0, 0, 0, 0);

    long long row0 = (((long long)blockIdx.x * 8 + warp) * ppw) * 2;
    bool valid = row0 < a.N;
    bool has2 = false;
    const uint4 *w0 = nullptr, *w1 = nullptr;
    uint4 c0[U], c1[U];

    auto fetch = [&](int cb, uint4* v0, uint4* v1) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int cc = cb + lane + 32 * u;
            const bool ok = cc < nch;
            v0[u] = ok ? ld_stream(w0 + cc) : zero;
            v1[u] = (ok && has2) ? ld_stream(w1 + cc) : zero;
        }
    };
    auto open_pair = [&]() {
        has2 = row0 + 1 < a.N;
        w0 = (const uint4*)((const WT*)a.W + row0 * a.K);
        w1 = w0 + nch;
        fetch(0, c0, c1);
    };
    if (valid) open_pair();          // the first weights are in flight while x is being staged

    load_x<WT, PRO>(a, b, xs, red);

    u64 best = 0;
    for (int pi = 0; valid;) {
        float acc0 = 0.f, acc1 = 0.f;
        for (int cb = 0; cb < nch; cb += 32 * U) {
            uint4 n0[U], n1[U];
            fetch(cb + 32 * U, n0, n1);
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int cc = cb + lane + 32 * u;
                if (cc < nch) {
                    if (sizeof(WT) == 2) {
                        const float4 xa = ((const float4*)xs)[cc];
                        const float4 xb = ((const float4*)(xs + (a.K >> 1)))[cc];
                        const uint4 p = c0[u], q = c1[u];
                        acc0 = fmaf(bf16_lo(p.x), xa.x, acc0); acc0 = fmaf(bf16_hi(p.x), xa.y, acc0);
                        acc0 = fmaf(bf16_lo(p.y), xa.z, acc0); acc0 = fmaf(bf16_hi(p.y), xa.w, acc0);
                        acc0 = fmaf(bf16_lo(p.z), xb.x, acc0); acc0 = fmaf(bf16_hi(p.z), xb.y, acc0);
                        acc0 = fmaf(bf16_lo(p.w), xb.z, acc0); acc0 = fmaf(bf16_hi(p.w), xb.w, acc0);
                        acc1 = fmaf(bf16_lo(q.x), xa.x, acc1); acc1 = fmaf(bf16_hi(q.x), xa.y, acc1);
                        acc1 = fmaf(bf16_lo(q.y), xa.z, acc1); acc1 = fmaf(bf16_hi(q.y), xa.w, acc1);
                        acc1 = fmaf(bf16_lo(q.z), xb.x, acc1); acc1 = fmaf(bf16_hi(q.z), xb.y, acc1);
                        acc1 = fmaf(bf16_lo(q.w), xb.z, acc1); acc1 = fmaf(bf16_hi(q.w), xb.w, acc1);
                    } else {
                        const float4 xa = ((const float4*)xs)[cc];
                        const uint4 p = c0[u], q = c1[u];
                        acc0 = fmaf(__uint_as_float(p.x), xa.x, acc0); acc0 = fmaf(__uint_as_float(p.y), xa.y, acc0);
                        acc0 = fmaf(__uint_as_float(p.z), xa.z, acc0); acc0 = fmaf(__uint_as_float(p.w), xa.w, acc0);
                        acc1 = fmaf(__uint_as_float(q.x), xa.x, acc1); acc1 = fmaf(__uint_as_float(q.y), xa.y, acc1);
                        acc1 = fmaf(__uint_as_float(q.z), xa.z, acc1); acc1 = fmaf(__uint_as_float(q.w), xa.w, acc1);
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) { c0[u] = n0[u]; c1[u] = n1[u]; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            acc0 += __shfl_xor_sync(0xffffffffu, acc0, o);
            acc1 += __shfl_xor_sync(0xffffffffu, acc1, o);
        }
        const long long done_row = row0;
        const bool done_has2 = has2;
        ++pi;
        row0 += 2;
        valid = pi < ppw && row0 < a.N;
        if (valid) open_pair();      // next pair's first loads go out before the stores below
        if (lane == 0) {
            float sq;
            u64 key = 0;
            epilogue_pair<WT, EPI>(a, b, (int)done_row, acc0, acc1, done_has2, 1.f, sq, key);
            best = key > best ? key : best;
        }
    }
    if (EPI == EPI_LM) {
        if (lane == 0) kred[warp] = best;
        __syncthreads();
        if (threadIdx.x == 0) {
            u64 m = kred[0];
#pragma unroll
            for (int w = 1; w < 8; ++w) m = kred[w] > m ? kred[w] : m;
            if (m) atomicMax(a.keys_out + (long long)b * a.keys_out_stride, m);
        }
    }
}

template <typename WT, int PRO, int EPI>
static cudaError_t launch_alu_t(const LinArgs& a, cudaStream_t st) {
    // the shared-memory opt-in is a per-device attribute of the function: remember it per device ordinal
    static bool attr_set[HIVIS_MAX_DEVICES] = {false};
    const size_t smem = (size_t)a.K * sizeof(float);
    int dev = 0;
    cudaError_t e0 = cudaGetDevice(&dev);
    if (e0 != cudaSuccess) return e0;
    if (dev < 0 || dev >= HIVIS_MAX_DEVICES || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(gemv_alu_kernel<WT, PRO, EPI>,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < HIVIS_MAX_DEVICES) attr_set[dev] = true;
    }
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    const long long pairs = ((long long)a.N + 1) / 2;
    int ppw = 1;                       // row pairs per warp: keep about 1000-2000 CTAs per launch
    while (ppw < 8 && pairs / (8LL * ppw * 2) >= 1184) ppw *= 2;
    const long long ctas = (pairs + 8LL * ppw - 1) / (8LL * ppw);
    dim3 grid((unsigned)ctas, (unsigned)a.B);
    gemv_alu_kernel<WT, PRO, EPI><<<grid, 256, smem, st>>>(a, ppw);
    return cudaGetLastError();
}

template <typename WT>
static cudaError_t launch_alu_d(int pro, int epi, const LinArgs& a, cudaStream_t st) {
    if (pro == PRO_FUSE && epi == EPI_FUSE) return launch_alu_t<WT, PRO_FUSE, EPI_FUSE>(a, st);
    if (pro == PRO_NORM && epi == EPI_QKV) return launch_alu_t<WT, PRO_NORM, EPI_QKV>(a, st);
    if (pro == PRO_PLAIN && epi == EPI_QKV) return launch_alu_t<WT, PRO_PLAIN, EPI_QKV>(a, st);
    if (pro == PRO_PLAIN && epi == EPI_OPROJ) return launch_alu_t<WT, PRO_PLAIN, EPI_OPROJ>(a, st);
    if (pro == PRO_NORM && epi == EPI_GATEUP) return launch_alu_t<WT, PRO_NORM, EPI_GATEUP>(a, st);
    if (pro == PRO_PLAIN && epi == EPI_DOWN) return launch_alu_t<WT, PRO_PLAIN, EPI_DOWN>(a, st);
    if (pro == PRO_PLAIN && epi == EPI_LM) return launch_alu_t<WT, PRO_PLAIN, EPI_LM>(a, st);
    return cudaErrorInvalidValue;
}

cudaError_t launch_gemv_alu(int dtype, int pro, int epi, const LinArgs& a, cudaStream_t st) {
    if (a.B <= 0 || a.N <= 0) return cudaSuccess;
    return dtype == HIVIS_BF16 ? launch_alu_d<bf16>(pro, epi, a, st) : launch_alu_d<float>(pro, epi, a, st);
}

// ==========================================================================================
// gemm_mma
// ==========================================================================================
__device__ __forceinline__ void mma_bf16(float (&c)[4], unsigned a0, unsigned a1, unsigned a2,
                                         unsigned a3, unsigned b0, unsigned b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int NI, int PRO, int EPI>
__global__ void __launch_bounds__(256) gemm_mma_kernel(const LinArgs a) {
    constexpr int MI = HIVIS_MMA_TILE_ROWS / 16;
    constexpr int U = 2;
    __shared__ float red[8][NI * 8][MI * 16 + 1];
    __shared__ float s_scale[NI * 8];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
    const long long row_base = (long long)blockIdx.x * (MI * 16);
    const int nch = a.K >> 3;
    const int nblk = (nch + 3) >> 2;
    const uint4 zero = make_uint4(0, 0, 0, 0);

    if (EPI == EPI_QKV || EPI == EPI_GATEUP) {
        if (tid < NI * 8) {
            float s = 1.f;
            if (tid < a.B) {
                float tot = 0.f;
                for (int i = 0; i < a.ssq_tiles; ++i) tot += __ldcg(a.ssq_in + (long long)i * a.ldb + tid);
                s = rsqrtf(tot / (float)a.K + a.eps);
            }
            s_scale[tid] = s;
        }
    }

    const uint4* wrow[MI][2];
    bool wok[MI][2];
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const long long r = row_base + mi * 16 + g + 8 * h;
            wok[mi][h] = r < a.N;
            wrow[mi][h] = (const uint4*)((const bf16*)a.W + (wok[mi][h] ? r : 0) * a.K);
        }
    // batch operand: row n = g + 8*ni; for PRO_FUSE the row is [feature ; embedding of its token]
    const uint4* xa[NI];
    const uint4* xb[NI];
    bool xok[NI];
    const int dch = a.d >> 3;
#pragma unroll
    for (int ni = 0; ni < NI; ++ni) {
        const int n = g + 8 * ni;
        xok[ni] = n < a.B;
        if (PRO == PRO_FUSE) {
            xa[ni] = (const uint4*)((const bf16*)a.feat_h + (long long)(xok[ni] ? n : 0) * a.d);
            const long long tok = xok[ni] ? fuse_token(a, n) : 0;
            xb[ni] = (const uint4*)((const bf16*)a.embed + tok * a.d);
        } else {
            xa[ni] = (const uint4*)(a.xin_h + (long long)(xok[ni] ? n : 0) * a.K);
            xb[ni] = xa[ni];
        }
    }

    float acc[MI][NI][4];
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
        for (int ni = 0; ni < NI; ++ni)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mi][ni][i] = 0.f;

    for (int blk = warp; blk < nblk; blk += 8 * U) {
        uint4 A[U][MI][2], X[U][NI];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int c = (blk + 8 * u) * 4 + t;
            const bool okc = c < nch;
#pragma unroll
            for (int mi = 0; mi < MI; ++mi)
#pragma unroll
                for (int h = 0; h < 2; ++h)
                    A[u][mi][h] = (okc && wok[mi][h]) ? ld_stream(wrow[mi][h] + c) : zero;
#pragma unroll
            for (int ni = 0; ni < NI; ++ni) {
                const uint4* p;
                if (PRO == PRO_FUSE) p = c < dch ? xa[ni] + c : xb[ni] + (c - dch);
                else p = xa[ni] + c;
                X[u][ni] = (okc && xok[ni]) ? ld_act(p) : zero;
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int mi = 0; mi < MI; ++mi)
#pragma unroll
                for (int ni = 0; ni < NI; ++ni) {
                    mma_bf16(acc[mi][ni], A[u][mi][0].x, A[u][mi][1].x, A[u][mi][0].y, A[u][mi][1].y,
                             X[u][ni].x, X[u][ni].y);
                    mma_bf16(acc[mi][ni], A[u][mi][0].z, A[u][mi][1].z, A[u][mi][0].w, A[u][mi][1].w,
                             X[u][ni].z, X[u][ni].w);
                }
    }
    // every warp holds a partial sum over its share of k: reduce across the 8 warps in fixed order
#pragma unroll
    for (int mi = 0; mi < MI; ++mi)
#pragma unroll
        for (int ni = 0; ni < NI; ++ni) {
            const int r = mi * 16 + g, bb = ni * 8 + 2 * t;
            red[warp][bb][r] = acc[mi][ni][0];
            red[warp][bb + 1][r] = acc[mi][ni][1];
            red[warp][bb][r + 8] = acc[mi][ni][2];
            red[warp][bb + 1][r + 8] = acc[mi][ni][3];
        }
    __syncthreads();
    constexpr int PAIRS = MI * 8;                  // 16 row pairs per tile
    if (tid < PAIRS * NI * 8) {
        const int b = tid / PAIRS, j = tid % PAIRS;
        float v0 = 0.f, v1 = 0.f;
#pragma unroll
        for (int w = 0; w < 8; ++w) {
            v0 += red[w][b][2 * j];
            v1 += red[w][b][2 * j + 1];
        }
        const long long row = row_base + 2 * j;
        const bool ok = b < a.B && row < a.N;
        float sq = 0.f;
        u64 key = 0;
        if (ok) {
            const float sc = (EPI == EPI_QKV || EPI == EPI_GATEUP) ? s_scale[b] : 1.f;
            epilogue_pair<bf16, EPI>(a, b, (int)row, v0, v1, row + 1 < a.N, sc, sq, key);
        }
        if ((EPI == EPI_FUSE || EPI == EPI_OPROJ) && a.ssq_out) {
#pragma unroll
            for (int o = PAIRS / 2; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
            if (j == 0 && b < a.B) a.ssq_out[(long long)blockIdx.x * a.ldb + b] = sq;
        }
        if (EPI == EPI_LM) {
#pragma unroll
            for (int o = PAIRS / 2; o > 0; o >>= 1) {
                const u64 other = __shfl_xor_sync(0xffffffffu, key, o);
                key = other > key ? other : key;
            }
            if (j == 0 && b < a.B && key) atomicMax(a.keys_out + (long long)b * a.keys_out_stride, key);
        }
    }
}

template <int NI>
static cudaError_t launch_mma_n(int pro, int epi, const LinArgs& a, cudaStream_t st) {
    const unsigned grid = (unsigned)((a.N + HIVIS_MMA_TILE_ROWS - 1) / HIVIS_MMA_TILE_ROWS);
#define HIVIS_MMA_CASE(P, E)                                    \
    if (pro == P && epi == E) {                                 \
        gemm_mma_kernel<NI, P, E><<<grid, 256, 0, st>>>(a);     \
        return cudaGetLastError();                              \
    }
    HIVIS_MMA_CASE(PRO_FUSE, EPI_FUSE)
    HIVIS_MMA_CASE(PRO_PLAIN, EPI_QKV)
    HIVIS_MMA_CASE(PRO_PLAIN, EPI_OPROJ)
    HIVIS_MMA_CASE(PRO_PLAIN, EPI_GATEUP)
    HIVIS_MMA_CASE(PRO_PLAIN, EPI_DOWN)
    HIVIS_MMA_CASE(PRO_PLAIN, EPI_LM)
#undef HIVIS_MMA_CASE
    return cudaErrorInvalidValue;
}

cudaError_t launch_gemm_mma(int pro, int epi, const LinArgs& a, cudaStream_t st) {
    if (a.B <= 0 || a.N <= 0) return cudaSuccess;
    if (a.B > 16) return cudaErrorInvalidValue;
    return a.B <= 8 ? launch_mma_n<1>(pro, epi, a, st) : launch_mma_n<2>(pro, epi, a, st);
}
