// Table precompute on the tensor cores: out[v] = W e_v + b for bf16 embeddings (text after Eq. 6: the projections depend only on the
// token id and are computed once).  This is the one dense contraction of the method, [V, E] x [E, m].
//
// The embeddings are bf16, hence exact as tensor-core operands; the fp32 weights are split into three bf16 parts,
// W = W1 + W2 + W3 (8 + 8 + 8 mantissa bits, the residual is below one fp32 ulp of W), and
//     out = bias + e W1^T + e W2^T + e W3^T
// is a bf16 GEMM with fp32 accumulation against the three parts side by side, [V, E] x [E, 3m], followed by the sum
// of the three column blocks: every product is exact in fp32, so the result differs from an fp32 GEMM only by the
// order of the additions.  The GEMM is a tcgen05 (UMMA) kernel with TMA operand loads and TMEM accumulators, built
// from the CUTLASS sm100 collective builders (128 x 128 x 64 tiles, one CTA per tile, no cluster, no multicast).
// It runs slab by slab over V (so that the fp32 partial sums of a slab stay in L2) and, within a slab, chunk by
// chunk over E (the accumulators of the tensor cores round less carefully than an FMA chain; the chunks' partial
// sums are added by the epilogue in plain fp32), so the embeddings are read from HBM once.
#include <cuda_runtime.h>

#include "cute/tensor.hpp"
#include "cutlass/cutlass.h"
#include "cutlass/epilogue/collective/collective_builder.hpp"
#include "cutlass/gemm/collective/collective_builder.hpp"
#include "cutlass/gemm/device/gemm_universal_adapter.h"
#include "cutlass/gemm/kernel/gemm_universal.hpp"
#include "cutlass/util/packed_stride.hpp"

#include "internal.h"

namespace graft {
namespace {

using ElementA = cutlass::bfloat16_t;  // embeddings [V, E], E contiguous
using ElementB = cutlass::bfloat16_t;  // one part of W [m, E], E contiguous = a column-major [E, m]
using ElementC = float;
using LayoutA = cutlass::layout::RowMajor;
using LayoutB = cutlass::layout::ColumnMajor;
using LayoutC = cutlass::layout::RowMajor;
constexpr int AlignA = 8, AlignB = 8, AlignC = 4;  // 16 bytes
using TileShape = cute::Shape<cute::_128, cute::_128, cute::_64>;
using ClusterShape = cute::Shape<cute::_1, cute::_1, cute::_1>;

using CollectiveEpilogue = typename cutlass::epilogue::collective::CollectiveBuilder<
    cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, TileShape, ClusterShape,
    cutlass::epilogue::collective::EpilogueTileAuto, float, float, ElementC, LayoutC, AlignC, ElementC, LayoutC, AlignC,
    cutlass::epilogue::collective::EpilogueScheduleAuto>::CollectiveOp;

using CollectiveMainloop = typename cutlass::gemm::collective::CollectiveBuilder<
    cutlass::arch::Sm100, cutlass::arch::OpClassTensorOp, ElementA, LayoutA, AlignA, ElementB, LayoutB, AlignB, float,
    TileShape, ClusterShape,
    cutlass::gemm::collective::StageCountAutoCarveout<static_cast<int>(sizeof(typename CollectiveEpilogue::SharedStorage))>,
    cutlass::gemm::collective::KernelScheduleAuto>::CollectiveOp;

using GemmKernel =
    cutlass::gemm::kernel::GemmUniversal<cute::Shape<int, int, int, int>, CollectiveMainloop, CollectiveEpilogue, void>;
using Gemm = cutlass::gemm::device::GemmUniversalAdapter<GemmKernel>;
#ifndef GRAFT_TABLES_CHUNK_K
#define GRAFT_TABLES_CHUNK_K 1024
#endif
constexpr int kTablesChunkK = GRAFT_TABLES_CHUNK_K;  // a multiple of 64 (the K extent of a tile)

// W (fp32, [m, E]) -> three bf16 parts; out rows <- bias
__global__ void weight_split_kernel(const float* __restrict__ W, size_t n, __nv_bfloat16* __restrict__ w1,
                                __nv_bfloat16* __restrict__ w2, __nv_bfloat16* __restrict__ w3) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const float w = W[i];
        const __nv_bfloat16 a = __float2bfloat16_rn(w);
        const float r1 = w - __bfloat162float(a);
        const __nv_bfloat16 b = __float2bfloat16_rn(r1);
        const float r2 = r1 - __bfloat162float(b);
        w1[i] = a;
        w2[i] = b;
        w3[i] = __float2bfloat16_rn(r2);
    }
}
// out[v][j] = bias[j] + tmp[v][j] + tmp[v][m + j] + tmp[v][2m + j] for the rows of one slab
__global__ void parts_reduce_kernel(const float* __restrict__ tmp, const float* __restrict__ bias, float* __restrict__ out,
                                 size_t rows, int m) {
    const size_t n = rows * (size_t)m;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const size_t v = i / m;
        const int j = (int)(i - v * m);
        const float* t = tmp + v * 3 * (size_t)m;
        out[i] = (bias ? bias[j] : 0.f) + ((t[j] + t[m + j]) + t[2 * (size_t)m + j]);
    }
}

}  // namespace

constexpr int kTablesSlabRows = 65536;  // rows of V per slab: 65536 x 3m fp32 partial sums (100 MB at m = 128), mostly L2-resident

// Scratch: three bf16 copies of W, a slab of partial sums, the GEMM's workspace.  Returns the bytes needed
// (0: this path cannot be used).
size_t tables_tc_scratch_bytes(int V, int E, int m) {
    if ((E % 8) != 0 || (m % 4) != 0 || V < 1) return 0;
    const int slab = V < kTablesSlabRows ? V : kTablesSlabRows;
    Gemm::Arguments args{cutlass::gemm::GemmUniversalMode::kGemm,
                         {slab, 3 * m, E, 1},
                         {nullptr, {}, nullptr, {}},
                         {{1.0f, 1.0f}, nullptr, {}, nullptr, {}}};
    const size_t ws = Gemm::get_workspace_size(args);
    return (((size_t)3 * m * E * sizeof(__nv_bfloat16) + 255) & ~(size_t)255) + (size_t)slab * 3 * m * sizeof(float) +
           ((ws + 255) & ~(size_t)255) + 512;
}

// out [V, m] = emb [V, E] (bf16) . W^T + bias on the tensor cores.  d_scratch: tables_tc_scratch_bytes, 256-byte aligned.
// Returns cudaErrorNotSupported when the GEMM cannot take the problem (the caller then uses the FMA kernel).
cudaError_t tables_tc_launch(const void* d_emb, int V, int E, int m, const float* d_W, const float* d_b, float* d_out,
                         void* d_scratch, int* launches, cudaStream_t st) {
    if (((uintptr_t)d_emb & 15) || ((uintptr_t)d_out & 15) || (E % 8) != 0 || (m % 4) != 0) return cudaErrorNotSupported;
    const int slab = V < kTablesSlabRows ? V : kTablesSlabRows;
    __nv_bfloat16* w3x = (__nv_bfloat16*)d_scratch;  // [3m, E]: W1 rows, then W2 rows, then W3 rows
    float* tmp = (float*)(((uintptr_t)(w3x + (size_t)3 * m * E) + 255) & ~(uintptr_t)255);  // [slab, 3m]
    void* ws = (void*)(((uintptr_t)(tmp + (size_t)slab * 3 * m) + 255) & ~(uintptr_t)255);
    weight_split_kernel<<<256, 256, 0, st>>>(d_W, (size_t)m * E, w3x, w3x + (size_t)m * E, w3x + (size_t)2 * m * E);
    *launches += 1;
    typename GemmKernel::StrideA sA{};
    typename GemmKernel::StrideB sB{};
    cute::get<0>(sA) = (int64_t)E;  // rows of the embeddings / of the W parts are E apart whatever the chunk
    cute::get<0>(sB) = (int64_t)E;
    for (int v0 = 0; v0 < V; v0 += slab) {
        const int rows = V - v0 < slab ? V - v0 : slab;
        auto sC = cutlass::make_cute_packed_stride(typename GemmKernel::StrideC{}, cute::make_shape(rows, 3 * m, 1));
        auto sD = cutlass::make_cute_packed_stride(typename GemmKernel::StrideD{}, cute::make_shape(rows, 3 * m, 1));
        for (int k0 = 0; k0 < E; k0 += kTablesChunkK) {
            const int kc = E - k0 < kTablesChunkK ? E - k0 : kTablesChunkK;
            Gemm::Arguments args{cutlass::gemm::GemmUniversalMode::kGemm,
                                 {rows, 3 * m, kc, 1},
                                 {(const ElementA*)d_emb + (size_t)v0 * E + k0, sA, (const ElementB*)w3x + k0, sB},
                                 {{1.0f, k0 == 0 ? 0.0f : 1.0f}, tmp, sC, tmp, sD}};
            Gemm gemm;
            if (gemm.can_implement(args) != cutlass::Status::kSuccess) return cudaErrorNotSupported;
            if (gemm.initialize(args, ws, st) != cutlass::Status::kSuccess) return cudaErrorUnknown;
            if (gemm.run(st) != cutlass::Status::kSuccess) return cudaErrorUnknown;
            *launches += 1;
        }
        parts_reduce_kernel<<<1024, 256, 0, st>>>(tmp, d_b, d_out + (size_t)v0 * m, (size_t)rows, m);
        *launches += 1;
    }
    return cudaGetLastError();
}

}  // namespace graft
