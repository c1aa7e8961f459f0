// cos(h_d, h_{d+1}) of two adjacent rows of the drafter's hidden states (Eq. 15), by one warp: fp64 accumulation,
// lanes stride the row.  Shared by the edge-score kernel's cosine CTAs and the tree kernel (when no edge-score
// kernel runs), so the SABA state has the same bits on both routes.
#pragma once
#include "common.cuh"

namespace graft {

// hidden: [rows, dh] bf16 or fp32; ra = element offset of row d (row d+1 follows it).  All lanes return the value.
__device__ __forceinline__ double warp_adjacent_cosine(const void* hidden, int hidden_bf16, int dh, size_t ra, int lane) {
    const size_t rb = ra + dh;
    double ab = 0.0, aa = 0.0, bb = 0.0;
    if (hidden_bf16 && (dh & 7) == 0 && ((uintptr_t)hidden & 15) == 0) {
        const uint4* pa = (const uint4*)((const uint16_t*)hidden + ra);
        const uint4* pb = (const uint4*)((const uint16_t*)hidden + rb);
        constexpr int CU = 4;  // vectors in flight per row and lane: the loads of a step are issued together
        for (int k0 = lane; k0 < dh / 8; k0 += 32 * CU) {
            uint4 va[CU], vb[CU];
#pragma unroll
            for (int u = 0; u < CU; ++u) {
                const int k = k0 + 32 * u;
                va[u] = k < dh / 8 ? pa[k] : make_uint4(0u, 0u, 0u, 0u);
                vb[u] = k < dh / 8 ? pb[k] : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < CU; ++u) {
                const uint32_t wa[4] = {va[u].x, va[u].y, va[u].z, va[u].w};
                const uint32_t wb[4] = {vb[u].x, vb[u].y, vb[u].z, vb[u].w};
                float fab = 0.f, faa = 0.f, fbb = 0.f;  // eight exact bf16 products per sum: fp32 is enough
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float x0 = __uint_as_float(wa[q] << 16), x1 = __uint_as_float(wa[q] & 0xFFFF0000u);
                    const float y0 = __uint_as_float(wb[q] << 16), y1 = __uint_as_float(wb[q] & 0xFFFF0000u);
                    fab = fmaf(x0, y0, fmaf(x1, y1, fab));
                    faa = fmaf(x0, x0, fmaf(x1, x1, faa));
                    fbb = fmaf(y0, y0, fmaf(y1, y1, fbb));
                }
                ab += (double)fab;
                aa += (double)faa;
                bb += (double)fbb;
            }
        }
    } else {
        for (int k = lane; k < dh; k += 32) {
            float x, y;
            if (hidden_bf16) {
                x = __uint_as_float(((uint32_t)((const uint16_t*)hidden)[ra + k]) << 16);
                y = __uint_as_float(((uint32_t)((const uint16_t*)hidden)[rb + k]) << 16);
            } else {
                x = ((const float*)hidden)[ra + k];
                y = ((const float*)hidden)[rb + k];
            }
            ab += (double)x * (double)y;
            aa += (double)x * (double)x;
            bb += (double)y * (double)y;
        }
    }
#pragma unroll
    for (int o2 = 16; o2 > 0; o2 >>= 1) {
        ab += __shfl_xor_sync(0xFFFFFFFFu, ab, o2);
        aa += __shfl_xor_sync(0xFFFFFFFFu, aa, o2);
        bb += __shfl_xor_sync(0xFFFFFFFFu, bb, o2);
    }
    return (aa > 0.0 && bb > 0.0) ? ab / (sqrt(aa) * sqrt(bb)) : 0.0;
}

}  // namespace graft
