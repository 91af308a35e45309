// Greedy verification for callers that must not allocate device memory.
//
// hivis_verify keeps its row-argmax keys in a buffer that hivis_init obtained from cudaMalloc.
// Some users of the library cannot make that call at all: a plug-in running inside a serving
// process whose memory pool already owns the whole GPU, code that runs while another component
// holds the allocator lock, or a host that forbids allocation once its start-up phase is over.
// For them the same two kernels are offered here with the keys in a fixed array that is part of
// the library image itself, so that nothing is allocated and no context is needed.
#include <mutex>

#include "hivis_internal.cuh"

void hivis_set_global_error(const char* msg);   // text later returned by hivis_last_error(NULL)

#define NOALLOC_ROWS (HIVIS_MAX_BATCH * (HIVIS_MAX_K + 1))
#define NOALLOC_CHUNK 8192   // logits per CTA
#define NOALLOC_MAX_DEVICES 64

// One packed (value, index) key per logits row.  Lives in every GPU that loads the library, from
// load until the process exits: 64 * 17 * 8 bytes = 8.5 KB.
static __device__ __align__(256) u64 g_noalloc_keys[NOALLOC_ROWS];

// Device addresses of the array, one per device, looked up on the first call made with that
// device current.  In host code the symbol itself is only a stand-in, never a device address.
static u64* g_keys_addr[NOALLOC_MAX_DEVICES];
static std::mutex g_keys_mutex;

template <typename LT>
__global__ void __launch_bounds__(256) noalloc_argmax_kernel(const void* logits, int V, u64* keys) {
    __shared__ u64 kred[8];
    const long long rowi = (long long)blockIdx.z * gridDim.y + blockIdx.y;   // b*(k+1) + j
    const LT* row = (const LT*)logits + rowi * V;
    const int c0 = blockIdx.x * NOALLOC_CHUNK;
    const int c1 = min(V, c0 + NOALLOC_CHUNK);
    constexpr int VEC = 16 / (int)sizeof(LT);
    u64 best = 0;
    // elements before the first 16-byte boundary of this chunk, then whole vectors, then the tail
    const size_t addr = (size_t)(row + c0);
    int head = (int)(((16 - (addr & 15)) & 15) / sizeof(LT));
    if (head > c1 - c0) head = c1 - c0;
    const int nvec = (c1 - c0 - head) / VEC;
    const uint4* rv = (const uint4*)(row + c0 + head);
    for (int i = threadIdx.x; i < nvec; i += 256) {
        const uint4 w = ld_stream(rv + i);
        const int e0 = c0 + head + i * VEC;
        float f[VEC];
        if constexpr (sizeof(LT) == 2) {
            f[0] = bf16_lo(w.x); f[1] = bf16_hi(w.x); f[2] = bf16_lo(w.y); f[3] = bf16_hi(w.y);
            f[4] = bf16_lo(w.z); f[5] = bf16_hi(w.z); f[6] = bf16_lo(w.w); f[7] = bf16_hi(w.w);
        } else {
            f[0] = __uint_as_float(w.x); f[1] = __uint_as_float(w.y);
            f[2] = __uint_as_float(w.z); f[3] = __uint_as_float(w.w);
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const u64 kk = pack_key(f[e], e0 + e);
            best = kk > best ? kk : best;
        }
    }
    for (int i = threadIdx.x; i < head; i += 256) {
        const u64 kk = pack_key(load_as_float<LT>(row, c0 + i), c0 + i);
        best = kk > best ? kk : best;
    }
    for (int i = c0 + head + nvec * VEC + threadIdx.x; i < c1; i += 256) {
        const u64 kk = pack_key(load_as_float<LT>(row, i), i);
        best = kk > best ? kk : best;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const u64 other = __shfl_xor_sync(0xffffffffu, best, o);
        best = other > best ? other : best;
    }
    if ((threadIdx.x & 31) == 0) kred[threadIdx.x >> 5] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
        u64 m = kred[0];
#pragma unroll
        for (int w = 1; w < 8; ++w) m = kred[w] > m ? kred[w] : m;
        if (m) atomicMax(keys + rowi, m);
    }
}

__global__ void noalloc_finish_kernel(int B, int k, const int32_t* draft_ids, const u64* keys,
                                      const int32_t* rows_before, int32_t* out_accept, int32_t* out_next,
                                      int32_t* out_kv_len) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const u64* kr = keys + (long long)b * (k + 1);
    int n = 0;
    while (n < k && key_index(kr[n]) == draft_ids[(long long)b * k + n]) ++n;
    out_accept[b] = n;
    out_next[b] = key_index(kr[n]);
    if (out_kv_len) out_kv_len[b] = rows_before[b] + 1 + (n < k - 1 ? n : k - 1);
}

static int noalloc_fail(int code, const char* msg) {
    hivis_set_global_error(msg);
    return code;
}

extern "C" int hivis_verify_noalloc(int B, int k, int vocab, const int32_t* draft_ids,
                                    const void* target_logits, int logits_dtype, const int32_t* rows_before,
                                    int32_t* out_accept, int32_t* out_next, int32_t* out_kv_len, void* stream) {
    if (B < 1 || B > HIVIS_MAX_BATCH)
        return noalloc_fail(HIVIS_ERR_CAPACITY, "hivis_verify_noalloc: B outside [1, HIVIS_MAX_BATCH]: the fixed key array holds HIVIS_MAX_BATCH * (HIVIS_MAX_K + 1) rows");
    if (k < 1 || k > HIVIS_MAX_K)
        return noalloc_fail(HIVIS_ERR_CAPACITY, "hivis_verify_noalloc: k outside [1, HIVIS_MAX_K]: the fixed key array holds HIVIS_MAX_BATCH * (HIVIS_MAX_K + 1) rows");
    if (vocab < 1) return noalloc_fail(HIVIS_ERR_SHAPE, "hivis_verify_noalloc: vocab must be positive");
    if (logits_dtype != HIVIS_F32 && logits_dtype != HIVIS_BF16)
        return noalloc_fail(HIVIS_ERR_DTYPE, "hivis_verify_noalloc: unknown logits dtype");
    if (!draft_ids || !target_logits || !out_accept || !out_next)
        return noalloc_fail(HIVIS_ERR_ARG, "hivis_verify_noalloc: null argument");
    if ((out_kv_len != nullptr) != (rows_before != nullptr))
        return noalloc_fail(HIVIS_ERR_ARG, "hivis_verify_noalloc: rows_before and out_kv_len must be given together");
    const void* ptrs[] = {draft_ids, target_logits, out_accept, out_next, rows_before, out_kv_len};
    for (const void* p : ptrs)
        if (p && (((uintptr_t)p) & 15u))
            return noalloc_fail(HIVIS_ERR_ARG, "hivis_verify_noalloc: device pointer not 16-byte aligned");

    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NOALLOC_MAX_DEVICES)
        return noalloc_fail(HIVIS_ERR_CUDA, "hivis_verify_noalloc: no usable current device");
    u64* keys = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_keys_mutex);
        if (!g_keys_addr[dev]) {       // first call on this device: ask the runtime where the array lives
            u64* p = nullptr;
            const cudaError_t e = cudaGetSymbolAddress((void**)&p, g_noalloc_keys);
            if (e != cudaSuccess || !p) {
                cudaGetLastError();
                return noalloc_fail(HIVIS_ERR_CUDA, "hivis_verify_noalloc: cudaGetSymbolAddress failed");
            }
            g_keys_addr[dev] = p;
        }
        keys = g_keys_addr[dev];
    }
    cudaStream_t st = (cudaStream_t)stream;
    // the array still holds the previous call's keys, and the argmax is an atomic max: clear it
    if (cudaMemsetAsync(keys, 0, sizeof(u64) * (size_t)B * (k + 1), st) != cudaSuccess)
        return noalloc_fail(HIVIS_ERR_CUDA, "hivis_verify_noalloc: clearing the key array failed");
    dim3 grid((unsigned)((vocab + NOALLOC_CHUNK - 1) / NOALLOC_CHUNK), (unsigned)(k + 1), (unsigned)B);
    if (logits_dtype == HIVIS_BF16) noalloc_argmax_kernel<bf16><<<grid, 256, 0, st>>>(target_logits, vocab, keys);
    else noalloc_argmax_kernel<float><<<grid, 256, 0, st>>>(target_logits, vocab, keys);
    if (cudaGetLastError() != cudaSuccess)
        return noalloc_fail(HIVIS_ERR_CUDA, "hivis_verify_noalloc: argmax kernel launch failed");
    noalloc_finish_kernel<<<1, 64, 0, st>>>(B, k, draft_ids, keys, rows_before, out_accept, out_next, out_kv_len);
    if (cudaGetLastError() != cudaSuccess)
        return noalloc_fail(HIVIS_ERR_CUDA, "hivis_verify_noalloc: finish kernel launch failed");
    return HIVIS_OK;
}
