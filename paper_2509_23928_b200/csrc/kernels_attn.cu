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
#include "attn_body.cuh"

template <typename WT, int DH, int GQ>
__global__ void __launch_bounds__(128) attn_decode_kernel(const AttnArgs a) {
    __shared__ AttnSmem<4, GQ, DH> sm;
    const int b = blockIdx.z;
    attn_unit<WT, DH, GQ, 4>(a, blockIdx.x, blockIdx.y, b, a.pos0[b] + a.step, a.slots[b], sm);
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
