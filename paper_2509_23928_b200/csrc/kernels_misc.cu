// Small kernels around the hot path: per-call state set-up, prefill bookkeeping, greedy
// verification with KV rollback, layout changes at init, debug read-back.
#include "attn_body.cuh"

// ------------------------------------------------------------------------------------------
// draft set-up / finish
// ------------------------------------------------------------------------------------------
__global__ void draft_setup_kernel(SlotList sl, int k, int d, int* d_slots, int* d_pos0, int* kv_len,
                                   const float* pend_feat, const int* pend_id, float* feat, bf16* feat_h,
                                   int* cur_id, u64* keys, int key_stride) {
    const int b = blockIdx.x, slot = sl.slot[b];
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
        feat_h[(long long)b * d + i] = __float2bfloat16_rn(v);
    }
}
cudaError_t launch_draft_setup(const SlotList& sl, int k, int d, int* d_slots, int* d_pos0,
                               int* kv_len, const float* pend_feat, const int* pend_id, float* feat,
                               bf16* feat_h, int* cur_id, u64* keys, int key_stride, cudaStream_t st) {
    draft_setup_kernel<<<sl.n, 256, 0, st>>>(sl, k, d, d_slots, d_pos0, kv_len, pend_feat, pend_id, feat,
                                             feat_h, cur_id, keys, key_stride);
    return cudaGetLastError();
}

__global__ void draft_finish_kernel(int n, int k, const u64* keys, int key_stride, int32_t* out_ids) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const int b = i / k, s = i % k;
    out_ids[i] = key_index(keys[(long long)b * key_stride + s]);
}
cudaError_t launch_draft_finish(int B, int k, const u64* keys, int key_stride, int32_t* out_ids,
                                cudaStream_t st) {
    const int n = B * k;
    draft_finish_kernel<<<(n + 127) / 128, 128, 0, st>>>(n, k, keys, key_stride, out_ids);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// type conversion
// ------------------------------------------------------------------------------------------
template <typename WT>
__global__ void convert_rows_kernel(const void* src, float* dst, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        dst[i] = load_as_float<WT>(src, i);
}
cudaError_t launch_convert_rows(int dtype, const void* src, float* dst, long long n, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const unsigned grid = (unsigned)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256);
    if (dtype == HIVIS_BF16) convert_rows_kernel<bf16><<<grid, 256, 0, st>>>(src, dst, n);
    else convert_rows_kernel<float><<<grid, 256, 0, st>>>(src, dst, n);
    return cudaGetLastError();
}
cudaError_t launch_bf16_to_f32(const bf16* src, float* dst, long long n, cudaStream_t st) {
    return launch_convert_rows(HIVIS_BF16, src, dst, n, st);
}
__global__ void f32_to_bf16_kernel(const float* src, bf16* dst, long long n) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n;
         i += (long long)gridDim.x * blockDim.x)
        dst[i] = __float2bfloat16_rn(src[i]);
}
cudaError_t launch_f32_to_bf16(const float* src, bf16* dst, long long n, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    const unsigned grid = (unsigned)((n + 255) / 256 > 1184 ? 1184 : (n + 255) / 256);
    f32_to_bf16_kernel<<<grid, 256, 0, st>>>(src, dst, n);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// prefill bookkeeping
// ------------------------------------------------------------------------------------------
template <typename WT>
__global__ void prefill_setup_kernel(SlotList sl, CuSeqlens cu, SlotList start, int d, const int32_t* ids,
                                     const void* hidden, int* kv_len, float* pend_feat, int* pend_id,
                                     int* slot_of, int* row_of) {
    __shared__ int s_base;
    const int b = blockIdx.x, slot = sl.slot[b];
    const int lo = cu.v[b], hi = cu.v[b + 1];
    if (threadIdx.x == 0) s_base = start.slot[b] >= 0 ? start.slot[b] : kv_len[slot];
    __syncthreads();
    const int base = s_base;
    for (int j = lo + threadIdx.x; j < hi; j += blockDim.x) {
        slot_of[j] = slot;
        row_of[j] = (j == hi - 1) ? -1 : base + (j - lo);
    }
    for (int i = threadIdx.x; i < d; i += blockDim.x)
        pend_feat[(long long)slot * d + i] = load_as_float<WT>(hidden, (long long)(hi - 1) * d + i);
    if (threadIdx.x == 0) {
        pend_id[slot] = ids[hi - 1];
        kv_len[slot] = base + (hi - lo) - 1;
    }
}
cudaError_t launch_prefill_setup(int dtype, const SlotList& sl, const CuSeqlens& cu, const SlotList& start,
                                 int d, const int32_t* ids, const void* hidden, int* kv_len,
                                 float* pend_feat, int* pend_id, int* slot_of, int* row_of,
                                 cudaStream_t st) {
    if (dtype == HIVIS_BF16)
        prefill_setup_kernel<bf16><<<sl.n, 256, 0, st>>>(sl, cu, start, d, ids, hidden, kv_len, pend_feat,
                                                         pend_id, slot_of, row_of);
    else
        prefill_setup_kernel<float><<<sl.n, 256, 0, st>>>(sl, cu, start, d, ids, hidden, kv_len, pend_feat,
                                                          pend_id, slot_of, row_of);
    return cudaGetLastError();
}

template <typename WT>
__global__ void kv_append_kernel(const float* kv, const int* slot_of, const int* row_of,
                                 const double* inv_freq, int Hkv, int dh, int max_len, void* Kc, void* Vc) {
    const int j = blockIdx.x;
    const int row = row_of[j];
    if (row < 0) return;
    const int slot = slot_of[j];
    const int half = dh / 2, kvw = Hkv * dh;
    const float* k = kv + (long long)j * 2 * kvw;
    const float* v = k + kvw;
    for (int i = threadIdx.x; i < Hkv * half; i += blockDim.x) {
        const int h = i / half, e = i % half;
        float c, s;
        rope_cs(row, inv_freq[e], c, s);
        const float x0 = k[h * dh + e], x1 = k[h * dh + e + half];
        const long long o = (((long long)slot * Hkv + h) * max_len + row) * dh;
        store_from_float<WT>(Kc, o + e, x0 * c - x1 * s);
        store_from_float<WT>(Kc, o + e + half, x1 * c + x0 * s);
    }
    for (int i = threadIdx.x; i < kvw; i += blockDim.x) {
        const int h = i / dh, e = i % dh;
        const long long o = (((long long)slot * Hkv + h) * max_len + row) * dh;
        store_from_float<WT>(Vc, o + e, v[i]);
    }
}
cudaError_t launch_kv_append(int dtype, const float* kv, int P, const int* slot_of, const int* row_of,
                             const double* inv_freq, int Hkv, int dh, int max_len, void* Kc, void* Vc,
                             cudaStream_t st) {
    if (P <= 0) return cudaSuccess;
    if (dtype == HIVIS_BF16)
        kv_append_kernel<bf16><<<P, 256, 0, st>>>(kv, slot_of, row_of, inv_freq, Hkv, dh, max_len, Kc, Vc);
    else
        kv_append_kernel<float><<<P, 256, 0, st>>>(kv, slot_of, row_of, inv_freq, Hkv, dh, max_len, Kc, Vc);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// greedy verification in one launch: row argmax over [B][k+1][V], accept length, next token, rollback
// ------------------------------------------------------------------------------------------
#define VERIFY_MAX_PASSES 8    // 16-byte loads a thread may have in flight
static_assert(HIVIS_MAX_K + 1 <= 32, "the finishing warp holds one row of a sequence per lane");

// One CTA per (chunk of a row, row, sequence); a chunk is `passes` x 256 16-byte vectors, all of a thread's loads
// issued before the first is used.  Every CTA folds its chunk into the row's packed argmax key (integer max:
// lowest index among equal values, independent of arrival order) and counts itself on the sequence's arrival
// counter; the CTA that completes the count reads the sequence's k + 1 keys and k draft ids (one per lane, so the
// loads overlap), finds the longest accepted prefix, writes the outputs, rolls the slot back, and leaves keys and
// counter zero for the next call.  Nobody waits.
template <typename LT>
__global__ void __launch_bounds__(256) verify_kernel(SlotList sl, int k, const void* logits, int V, int passes,
                                                     const int32_t* draft_ids, u64* keys, int* arrivals,
                                                     int* kv_len, int32_t* out_accept, int32_t* out_next,
                                                     int32_t* out_kv_len) {
    __shared__ u64 kred[8];
    constexpr int VEC = 16 / (int)sizeof(LT);
    const int b = blockIdx.z;
    const long long rowi = (long long)b * (k + 1) + blockIdx.y;
    const LT* row = (const LT*)logits + rowi * V;
    const int chunk = passes * 256 * VEC;
    const int c0 = blockIdx.x * chunk;
    const int c1 = min(V, c0 + chunk);
    u64 best = 0;
    const bool aligned = (((size_t)(row + c0)) & 15) == 0;
    if (aligned) {
        const int nvec = (c1 - c0) / VEC;                 // <= passes * 256
        const uint4* rv = (const uint4*)(row + c0);
        uint4 w[VERIFY_MAX_PASSES];
#pragma unroll
        for (int p = 0; p < VERIFY_MAX_PASSES; ++p) {
            const int i = threadIdx.x + p * 256;
            if (i < nvec) w[p] = ld_stream(rv + i);
        }
#pragma unroll
        for (int p = 0; p < VERIFY_MAX_PASSES; ++p) {
            const int i = threadIdx.x + p * 256;
            if (i < nvec) {
                const int e0 = c0 + i * VEC;
                float f[VEC];
                if constexpr (sizeof(LT) == 2) {
                    f[0] = bf16_lo(w[p].x); f[1] = bf16_hi(w[p].x); f[2] = bf16_lo(w[p].y); f[3] = bf16_hi(w[p].y);
                    f[4] = bf16_lo(w[p].z); f[5] = bf16_hi(w[p].z); f[6] = bf16_lo(w[p].w); f[7] = bf16_hi(w[p].w);
                } else {
                    f[0] = __uint_as_float(w[p].x); f[1] = __uint_as_float(w[p].y);
                    f[2] = __uint_as_float(w[p].z); f[3] = __uint_as_float(w[p].w);
                }
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const u64 kk = pack_key(f[e], e0 + e);
                    best = kk > best ? kk : best;
                }
            }
        }
        for (int i = c0 + nvec * VEC + threadIdx.x; i < c1; i += 256) {       // V not a multiple of the vector
            const u64 kk = pack_key(load_as_float<LT>(row, i), i);
            best = kk > best ? kk : best;
        }
    } else {
        for (int i = c0 + threadIdx.x; i < c1; i += 256) {
            const u64 kk = pack_key(load_as_float<LT>(row, i), i);
            best = kk > best ? kk : best;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((threadIdx.x & 31) == 0) kred[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    int last = 0;
    if (lane == 0) {
        u64 m = kred[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) m = kred[w] > m ? kred[w] : m;
        atomicMax(keys + rowi, m);
        // release: the key update above is visible before the count; acquire: so are those of earlier arrivers
        const int total = (int)gridDim.x * (k + 1);
        last = atom_add_acq_rel(arrivals + b, 1) == total - 1;
    }
    if (!__shfl_sync(0xffffffffu, last, 0)) return;
    // lane j holds row j of the sequence: its argmax and the draft token it is compared with
    u64* kr = keys + (long long)b * (k + 1);
    const int slot = sl.slot[b];
    const int len = kv_len[slot];
    const int am = lane <= k ? key_index(__ldcg(kr + lane)) : 0;
    const int dj = lane < k ? draft_ids[(long long)b * k + lane] : -1;
    const unsigned miss = __ballot_sync(0xffffffffu, lane < k && am != dj);
    const int n = miss ? __ffs(miss) - 1 : k;             // length of the accepted prefix
    const int next = __shfl_sync(0xffffffffu, am, n);
    if (lane <= k) kr[lane] = 0ull;
    if (lane != 0) return;
    const int pairs = len - k + 1;                        // true-feature pairs of the sequence
    const int rows = pairs + (n < k - 1 ? n : k - 1);
    kv_len[slot] = rows;
    out_accept[b] = n;
    out_next[b] = next;
    if (out_kv_len) out_kv_len[b] = rows;
    arrivals[b] = 0;
}

cudaError_t launch_verify(int logits_dtype, const SlotList& sl, int k, int V, const int32_t* draft_ids,
                          const void* logits, u64* keys, int* arrivals, int* kv_len, int32_t* out_accept,
                          int32_t* out_next, int32_t* out_kv_len, cudaStream_t st, int* n_launches) {
    // the shortest chunk that still puts every CTA on the device at once (148 SMs x 8 CTAs of 256 threads)
    const int per_pass = 256 * (logits_dtype == HIVIS_BF16 ? 8 : 4);
    const long long rows = (long long)sl.n * (k + 1);
    int passes = 1;
    while (passes < VERIFY_MAX_PASSES && rows * ((V + passes * per_pass - 1) / (passes * per_pass)) > 148 * 8) ++passes;
    const int chunk = passes * per_pass;
    dim3 grid((unsigned)((V + chunk - 1) / chunk), (unsigned)(k + 1), (unsigned)sl.n);
    if (logits_dtype == HIVIS_BF16)
        verify_kernel<bf16><<<grid, 256, 0, st>>>(sl, k, logits, V, passes, draft_ids, keys, arrivals, kv_len,
                                                   out_accept, out_next, out_kv_len);
    else
        verify_kernel<float><<<grid, 256, 0, st>>>(sl, k, logits, V, passes, draft_ids, keys, arrivals, kv_len,
                                                    out_accept, out_next, out_kv_len);
    *n_launches = 1;
    return cudaGetLastError();
}

__global__ void set_int_kernel(int* p, int v) { *p = v; }
__global__ void set_rows_kernel(SlotList sl, CuSeqlens rows, int* kv_len) {
    if ((int)threadIdx.x < sl.n) kv_len[sl.slot[threadIdx.x]] = rows.v[threadIdx.x];
}
cudaError_t launch_set_rows(const SlotList& sl, const CuSeqlens& rows, int* kv_len, cudaStream_t st) {
    set_rows_kernel<<<1, HIVIS_MAX_BATCH, 0, st>>>(sl, rows, kv_len);
    return cudaGetLastError();
}
cudaError_t launch_set_int(int* p, int v, cudaStream_t st) {
    set_int_kernel<<<1, 1, 0, st>>>(p, v);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------
// init-time layout change: copy `rows` rows of row_bytes bytes to rows dst_row0 + r*dst_row_step
// ------------------------------------------------------------------------------------------
__global__ void copy_rows_kernel(const uint4* src, uint4* dst, long long rows, long long vec_per_row,
                                 long long dst_row0, long long dst_row_step) {
    const long long total = rows * vec_per_row;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long r = i / vec_per_row, c = i % vec_per_row;
        dst[(dst_row0 + r * dst_row_step) * vec_per_row + c] = src[i];
    }
}
cudaError_t launch_copy_rows(const void* src, void* dst, long long rows, long long row_bytes,
                             long long dst_row0, long long dst_row_step, cudaStream_t st) {
    if (rows <= 0) return cudaSuccess;
    if (row_bytes % 16) return cudaErrorInvalidValue;
    copy_rows_kernel<<<1184, 256, 0, st>>>((const uint4*)src, (uint4*)dst, rows, row_bytes / 16, dst_row0,
                                           dst_row_step);
    return cudaGetLastError();
}

template <typename WT>
__global__ void read_kv_kernel(const void* Kc, const void* Vc, int slot, int row0, int n, int Hkv, int dh,
                               int max_len, float* out_k, float* out_v) {
    const long long total = (long long)n * Hkv * dh;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int e = (int)(i % dh);
        const int h = (int)((i / dh) % Hkv);
        const int r = (int)(i / ((long long)dh * Hkv));
        const long long o = (((long long)slot * Hkv + h) * max_len + row0 + r) * dh + e;
        out_k[i] = load_as_float<WT>(Kc, o);
        out_v[i] = load_as_float<WT>(Vc, o);
    }
}
cudaError_t launch_read_kv(int dtype, const void* Kc, const void* Vc, int slot, int row0, int n, int Hkv,
                           int dh, int max_len, float* out_k, float* out_v, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    if (dtype == HIVIS_BF16)
        read_kv_kernel<bf16><<<256, 256, 0, st>>>(Kc, Vc, slot, row0, n, Hkv, dh, max_len, out_k, out_v);
    else
        read_kv_kernel<float><<<256, 256, 0, st>>>(Kc, Vc, slot, row0, n, Hkv, dh, max_len, out_k, out_v);
    return cudaGetLastError();
}
