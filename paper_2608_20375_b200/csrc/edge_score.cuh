// TDES edge scores of one depth out of shared memory (Eq. 4-6), shared by the edge-score kernel (which scores the
// first depths for every sequence) and the tree kernel (which scores deeper depths when an expansion gets there),
// so that a row has the same bits whichever kernel produced it.
//
//   f[p][c]    = s/sqrt(m) * (P[p] + u_d) . (C[c] + u_d)                                   (Eq. 4-6)
//   edge[p][c] = log q_d(c) + beta * (f[p][c] - mean_c f[p][c])                            (TDES score)
//   and every parent's row ordered by (edge descending, child rank ascending).
#pragma once
#include "common.cuh"

namespace graft {

// Will this sequence's tree run deep?  A confident drafter (high top-1 probabilities) gives a deep, narrow tree that
// needs the edge scores of many depths; an uncertain one a shallow, wide tree that stops a few levels down.  The
// edge-score kernel scores the deeper rows ahead of the tree kernel only for the sequences that pass this test (mean
// top-1 probability of the block >= 0.2: on the configured workloads trees reach depth 8 from about there); the tree
// kernel, which takes the same decision from the same numbers, scores what is missing on demand.  A matter of speed
// only: a row has the same bits whoever scores it.
// (In two steps, so that a caller can have the load in flight beside its other loads: lane d's top-1 log-probability
// of position d, 0 for d >= L; then the decision, taken by every lane of a warp together.)
__device__ __forceinline__ float deep_tree_load(const float* __restrict__ topk_lp_seq, int L, int K) {
    const int lane = threadIdx.x & 31;
    return lane < L ? topk_lp_seq[(size_t)lane * K] : 0.f;
}
__device__ __forceinline__ bool deep_tree_decide(float lp_top, int L) {
    // lane d holds position d (L <= 32); a butterfly sum in a fixed order
    const int lane = threadIdx.x & 31;
    float s = lane < L ? ex2_approx(lp_top * kLog2e) : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, o);
    return s >= 0.2f * (float)L;
}
__device__ __forceinline__ bool deep_tree_likely(const float* __restrict__ topk_lp_seq, int L, int K) {
    return deep_tree_decide(deep_tree_load(topk_lp_seq, L, K), L);
}


// Where the r-th entry of the sorted row of parent rank c stands inside the row (scores only; the child ranks stand
// in order): rotated by the parent's rank.  The tree kernel's threads look at the same place r of different parents'
// rows far more often than at different places of one row, and with K = 32 a row is one pass over the shared-memory
// banks: unrotated, such a look is a 32-way bank conflict.
__device__ __forceinline__ int es_col(int r, int c, int K) {
    const int x = r + c;
    return x < K ? x : x - K;
}

// K x K dot products by 8 warps.  Warp ty takes parents ty, ty+8, ty+16, ty+24; lane = (ks, tx): children tx and
// tx+16, and every second float4 of the m axis starting at ks.  A lane keeps a 4 x 2 tile of running sums, each as
// a packed fp32 pair (even and odd elements of the m axis; `fma.rn.f32x2`, so 16 packed FMAs per six 16-byte
// loads); the pair is added at the end and the two ks of a tile by one butterfly step, in a fixed order.
// rP / rC: [.][ld] rows in shared memory, ld = m + 4 floats (16-byte aligned, conflict-free float4 reads).
// ADD_U: the rows hold P and C and u is added on the way into the registers; otherwise they already hold P + u and
// C + u (the same fp32 sums either way).  part: [K][K] floats of shared memory; rows >= n_par are not written.
template <bool ADD_U>
__device__ __forceinline__ void edge_dots(const float* rP, const float* rC, const float* rU, int m, int K, int n_par,
                                          float* part, int ty, int lane) {
    if (ty >= n_par) return;
    const int tx = lane & 15, ks = lane >> 4, q4 = m / 4, ld = m + 4;
    float2 acc[4][2];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int i2 = 0; i2 < 2; ++i2) acc[i][i2] = make_float2(0.f, 0.f);
    const float* c0 = rC + (size_t)min(tx, K - 1) * ld;  // (rows past K: read, never used)
    const float* c1 = rC + (size_t)min(tx + 16, K - 1) * ld;
#pragma unroll 2
    for (int k4 = ks; k4 < q4; k4 += 2) {
        float4 uu = make_float4(0.f, 0.f, 0.f, 0.f);
        if (ADD_U) uu = *(const float4*)(rU + 4 * k4);
        float4 cv[2];
        cv[0] = *(const float4*)(c0 + 4 * k4);
        cv[1] = *(const float4*)(c1 + 4 * k4);
        if (ADD_U) {
#pragma unroll
            for (int i2 = 0; i2 < 2; ++i2) {
                cv[i2].x += uu.x;
                cv[i2].y += uu.y;
                cv[i2].z += uu.z;
                cv[i2].w += uu.w;
            }
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float4 pv = *(const float4*)(rP + (size_t)min(ty + 8 * i, n_par - 1) * ld + 4 * k4);
            if (ADD_U) {
                pv.x += uu.x;
                pv.y += uu.y;
                pv.z += uu.z;
                pv.w += uu.w;
            }
#pragma unroll
            for (int i2 = 0; i2 < 2; ++i2) {
                float2 a = acc[i][i2];
                a = __ffma2_rn(make_float2(pv.x, pv.y), make_float2(cv[i2].x, cv[i2].y), a);
                a = __ffma2_rn(make_float2(pv.z, pv.w), make_float2(cv[i2].z, cv[i2].w), a);
                acc[i][i2] = a;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        float v[2];
#pragma unroll
        for (int i2 = 0; i2 < 2; ++i2) {
            float a = acc[i][i2].x + acc[i][i2].y;
            a += __shfl_xor_sync(0xFFFFFFFFu, a, 16);
            v[i2] = a;
        }
        if (ks == (i & 1) && ty + 8 * i < n_par) {
            if (tx < K) part[(size_t)(ty + 8 * i) * K + tx] = v[0];
            if (tx + 16 < K) part[(size_t)(ty + 8 * i) * K + tx + 16] = v[1];
        }
    }
}

// One warp finishes one parent's row: scale, centre over the K children, add log q (lane = child c), and find the
// place of every child in the order (edge descending, child rank ascending) by counting the children that come
// before it.  dots: the parent's K dot products, or nullptr for a parent that does not exist (a row of zeros).
// wsc: 32 words of shared memory of this warp.  Returns the score in `val` and the place in `rank` (lanes < K).
__device__ __forceinline__ void edge_row_finish(const float* dots, const float* lps, float scale, float beta, int K,
                                                float inv_K, uint32_t* wsc, int lane, float& val, int& rank) {
    const int c = lane;
    val = 0.f;
    if (dots != nullptr) {
        const float ft = c < K ? dots[c] * scale : 0.f;
        float sum = ft;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, d);
        // sum / K: the product with 1 / K (worked out once by the caller) and one correction step with the exact
        // remainder, which gives the rounded quotient without the division's special-case code
        const float q0 = sum * inv_K;
        const float mean = fmaf(fmaf(-q0, (float)K, sum), inv_K, q0);
        val = fmaf(beta, ft - mean, c < K ? lps[c] : 0.f);
    }
    const uint32_t mine = c < K ? ord_from_float(val) : 0u;  // 0 is below the image of every float
    __syncwarp();
    wsc[c] = mine;
    __syncwarp();
    rank = 0;
#pragma unroll
    for (int i4 = 0; i4 < 8; ++i4) {
        const uint4 o4 = *(const uint4*)(wsc + 4 * i4);
        rank += (o4.x > mine ? 1 : 0) + (o4.y > mine ? 1 : 0) + (o4.z > mine ? 1 : 0) + (o4.w > mine ? 1 : 0);
    }
    // equal scores (rare) go by child rank: the counts above are a permutation of 0..K-1 unless some scores are equal,
    // and only then are the lanes with the same score looked up (a slow instruction)
    const uint32_t seen = __reduce_or_sync(0xFFFFFFFFu, c < K ? 1u << rank : 0u);
    if (seen != (K == 32 ? 0xFFFFFFFFu : (1u << K) - 1u)) {  // (uniform)
        const uint32_t same = __match_any_sync(0xFFFFFFFFu, mine);
        rank += __popc(same & ((1u << lane) - 1u));
    }
}

}  // namespace graft
