// Vocab pass: for every (sequence, future position) row of the drafter logits, one streaming read that
// yields log-sum-exp over the vocabulary and the K top-ranked tokens with their log-probabilities
// (Preliminaries, "DFlash one-pass marginals": q_{t,d} and c^{(r)}_{t,d}; Eq. 3's log q).
//
// Shape of the kernel (sm_100a):
//   * persistent grid, one CTA per SM; the rows*V element stream is cut into equal contiguous shares,
//     one per CTA, so a CTA sees at most two partial rows plus whole rows in between ("segments");
//   * warp roles: one producer warp feeds a four-stage shared-memory ring with 32 KiB TMA bulk copies
//     (cp.async.bulk + mbarrier complete_tx); sixteen streaming warps read the ring with 16-byte shared loads;
//     two epilogue groups of four warps finish alternate segments while the streaming warps are already in
//     later ones; one warp computes the adjacent-position cosines of the SABA state (Eq. 15) beside the stream;
//   * per 32-element chunk a streaming lane takes a packed max (stored for the second stage, 2 bytes per
//     chunk), keeps a lazily rescaled reference exponent and adds 2^(z log2e - ref) with ex2.approx;
//   * top-K needs no per-element work in the stream: after the segment, the K-th largest of 64 group maxima
//     is a lower bound T for the K-th largest element; only chunks whose stored max reaches T
//     (about K of them) are re-read, their elements >= T become 64-bit keys (value desc, id asc) and the
//     exact top-K is found by rank counting.  Rows that defeat the bound: when more chunks reach T than the
//     hit list holds, T is raised to the K-th largest chunk maximum (or, where the group maxima tie, the
//     elements above T and the first ones equal to T are taken); hundreds of keys are selected by a search
//     over the key's bits instead of ranked; an overflow of the key buffer falls back to an exact selection
//     over the segment whose filter starts at T;
//   * rows shared by several CTAs are merged by the last CTA to arrive (a counter, no waiting);
//   * vocabulary-parallel use: the row's pieces are left for a merge over shards instead (vocab_merge_kernel).
// Every wait on an mbarrier is bounded; when one runs out the kernel raises an error flag and drains.
#include <stdlib.h>
#include <string.h>

#include <mutex>

#include "common.cuh"
#include "internal.h"
#include "cosine.cuh"

#ifndef GRAFT_VP_F32X2
#define GRAFT_VP_F32X2 1  // packed fp32 pair arithmetic (fma.rn.f32x2 / add.rn.f32x2)
#endif

namespace graft {

namespace {


constexpr int NW = kVpConsumerWarps;          // streaming warps
constexpr int NT = kVpConsumers;              // streaming threads
constexpr int PROD_WARP = NW + kVpEpiGroups * kVpEpiThreads / 32;  // warp index of the producer warp
constexpr int TILE = kVpTileBytes;
constexpr int WBLK = TILE / NW;               // bytes of a tile owned by one warp (2048)
static_assert(WBLK == 2048, "one warp owns 2 KiB of every tile");
constexpr int VEC_PER_LANE = WBLK / 16 / 32;  // 4
static_assert(VEC_PER_LANE == 4, "chunk layout assumes four 16-byte vectors per lane per tile");
static_assert(WBLK == 32 * 4 * 16, "the exact fall-back selection reads one warp block per batch");
constexpr uint32_t kOrdNegInf = 0x007FFFFFu;  // ord_from_bits of -inf: every finite value maps above it
constexpr uint32_t kVpIdleHintNs = 10000;  // suspend hint of the waits of the producer and epilogue warps
constexpr int COS_WARP = PROD_WARP + 1;  // warp that computes the SABA cosines beside the stream
static_assert(kVpThreads == NT + kVpEpiGroups * kVpEpiThreads + 64,
              "thread count = streaming warps + epilogue warps + producer warp + cosine warp");

template <bool BF16>
struct VT;
template <>
struct VT<true> {
    using cm_t = uint16_t;
    static constexpr int ESZ = 2, EPV = 8;
    static constexpr uint32_t NEG_INF_WORD = 0xFF80FF80u;
};
template <>
struct VT<false> {
    using cm_t = uint16_t;  // the chunk maximum rounded UP to bf16 precision: an upper bound is all the scan needs
    static constexpr int ESZ = 4, EPV = 4;
    static constexpr uint32_t NEG_INF_WORD = 0xFF800000u;
};

struct VpParams {
    const char* logits;
    int rows, V, K;
    long long nq;  // quanta per row
    long long Q;   // quanta in total
    int stages;
    int n_cmax;    // chunk-max slots per buffer (two buffers): 256 threads x max_tiles
    int max_tiles; // slots per streaming thread
    VpRecord* records;
    int* row_counter;
    int32_t* topk_id;
    float* topk_lp;
    float* lse;
    int32_t* row_status;
    int32_t* errflag;
    graft_vocab_partial* partial_out;  // vocabulary-parallel use: the row's pieces go here instead of the outputs
    // adjacent-position cosines of the SABA state (Eq. 15), computed by a warp of their own beside the stream;
    // cos_out == nullptr: not asked for
    const void* hidden;
    int hidden_bf16, hidden_dim, L;
    double* cos_out;  // [rows / L, L]
    int use_hint;
};

struct Seg {
    int row, e0, e1;
    const char* body;
    uint32_t body_bytes;
    int e_body0, e_tail0;
    int ntiles;
};

__device__ __forceinline__ long long cta_start(long long g, long long Q, long long G) { return g * Q / G; }
__device__ __forceinline__ int cta_of(long long x, long long Q, long long G) {
    return (int)(((x + 1) * G + Q - 1) / Q - 1);
}

// The piece [qr0, qr1) (in quanta) of row `row`.  No division: segment boundaries are on the streaming warps' path.
template <bool BF16>
__device__ __forceinline__ Seg make_seg(const VpParams& p, int row, int qr0, int qr1) {
    using T = VT<BF16>;
    Seg s;
    s.row = row;
    s.e0 = qr0 * kVpQuantum;
    s.e1 = qr1 == (int)p.nq ? p.V : qr1 * kVpQuantum;  // the last quantum of a row also takes the remainder
    const char* a0 = p.logits + ((size_t)s.row * p.V + s.e0) * T::ESZ;
    const char* a1 = p.logits + ((size_t)s.row * p.V + s.e1) * T::ESZ;
    uintptr_t b0 = ((uintptr_t)a0 + 15) & ~(uintptr_t)15;
    uintptr_t b1 = (uintptr_t)a1 & ~(uintptr_t)15;
    if (b1 < b0) b1 = b0;
    if (b0 > (uintptr_t)a1) {  // the segment holds no 16-byte aligned address at all
        b0 = b1 = (uintptr_t)a1;
    }
    s.body = (const char*)b0;
    s.body_bytes = (uint32_t)(b1 - b0);
    s.e_body0 = s.e0 + (int)((b0 - (uintptr_t)a0) / T::ESZ);
    s.e_tail0 = s.e_body0 + (int)(s.body_bytes / T::ESZ);
    s.ntiles = (int)((s.body_bytes + TILE - 1) / TILE);
    return s;
}

// A CTA's share of the stream as a list of segments.  The share's last segment (usually a partial row that is
// shared with the next CTA) is visited FIRST, so that the cross-CTA merge of shared rows happens early instead
// of at the kernel's tail; the remaining segments follow in stream order.  Two divisions when the walk begins, none
// per segment.
struct SegIter {
    int r_first, r_last;  // rows of the share's first and last quantum
    int qr_first;         // where the share begins within r_first
    int qr_last0, qr_last1;  // the last segment's piece of r_last
    int row;              // next row of the walk over [r_first, r_last)
    int state;            // 0: emit the last segment, 1: walk, 2: nothing at all
    bool whole_last;      // the last segment is the only one (it starts where the share starts)
};
template <bool BF16>
__device__ __forceinline__ SegIter seg_iter_begin(const VpParams& p, long long q0, long long q1) {
    SegIter it;
    it.state = q0 < q1 ? 0 : 2;
    it.r_first = (int)(q0 / p.nq);
    it.qr_first = (int)(q0 - (long long)it.r_first * p.nq);
    it.r_last = (int)((q1 - 1) / p.nq);
    // the last segment starts at the last row boundary inside the share (or where the share starts)
    it.whole_last = it.r_last == it.r_first;
    it.qr_last0 = it.whole_last ? it.qr_first : 0;
    it.qr_last1 = (int)(q1 - (long long)it.r_last * p.nq);
    it.row = it.r_first;
    return it;
}
template <bool BF16>
__device__ __forceinline__ bool seg_iter_next(const VpParams& p, SegIter& it, Seg& sg) {
    if (it.state == 0) {
        sg = make_seg<BF16>(p, it.r_last, it.qr_last0, it.qr_last1);
        it.state = 1;
        return true;
    }
    if (it.state == 2 || it.row >= it.r_last) return false;
    sg = make_seg<BF16>(p, it.row, it.row == it.r_first ? it.qr_first : 0, (int)p.nq);
    ++it.row;
    return true;
}
// After seg_iter_next returned a segment: is it the one this CTA visits last?
__device__ __forceinline__ bool seg_iter_at_end(const SegIter& it) { return it.row >= it.r_last; }

__device__ __forceinline__ float load_elem_f32(const char* p, bool bf16) {
    if (bf16) return __uint_as_float(((uint32_t) * (const uint16_t*)p) << 16);
    return *(const float*)p;
}

// ---- per-thread streaming state -----------------------------------------------------------------
#if GRAFT_VP_F32X2
__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
#endif

// The running log-sum-exp of one streaming thread over a segment: sum of 2^(z log2e - ref) in four fp32
// accumulators (two packed pairs), a reference exponent that is raised lazily (only when a chunk's maximum exceeds
// it by more than 2^16, so that rescaling is rare and every term stays far from overflow), and the largest value.
struct Acc {
    float ref;      // reference exponent, log2 domain; -inf before the first finite value
    float nref;     // -ref (0 while ref is -inf): the addend of the fused multiply-add
    uint32_t thr;   // a chunk maximum above this value raises the reference: bf16 logits: the value in both halves
                    // of a packed pair; fp32 logits: float bits
    uint32_t rmax;  // largest value so far: bf16 logits: a packed pair of running maxima; fp32 logits: float bits
#if GRAFT_VP_F32X2
    uint64_t a0, a1;
#else
    float s0, s1, s2, s3;
#endif
};

template <bool BF16>
__device__ __forceinline__ void acc_init(Acc& a) {
    a.ref = -INFINITY;
    a.nref = 0.f;
    a.thr = BF16 ? 0xFF80FF80u : 0xFF800000u;  // -inf: the first finite value sets the reference
    a.rmax = a.thr;
#if GRAFT_VP_F32X2
    a.a0 = a.a1 = 0ull;
#else
    a.s0 = a.s1 = a.s2 = a.s3 = 0.f;
#endif
}

// The chunk maximum cm exceeded the threshold: raise the reference to cm (rare).
template <bool BF16>
__device__ __forceinline__ void acc_raise(Acc& a, float cm) {
    const float cms = cm * kLog2e;
    if (!(cms > a.ref + 16.0f)) return;  // (the threshold is a truncated copy of ref + 16: it may fire a little early)
    const float f = ex2_approx(a.ref - cms);  // 0 when ref is -inf (nothing added yet) or cm is +inf
#if GRAFT_VP_F32X2
    const uint64_t f2 = pack2(f, f);
    a.a0 = mul2(a.a0, f2);
    a.a1 = mul2(a.a1, f2);
#else
    a.s0 *= f;
    a.s1 *= f;
    a.s2 *= f;
    a.s3 *= f;
#endif
    a.ref = cms;
    a.nref = -cms;
    // values above (ref + 16) / log2e raise the reference again; the bound need not be exact (terms overflow only
    // 2^111 above it), so it is kept as its leading 16 bits for the packed comparison of bf16 chunks
    const uint32_t zb = __float_as_uint((cms + 16.0f) * 0.6931471805599453f);
    a.thr = BF16 ? ((zb >> 16) | (zb & 0xFFFF0000u)) : zb;
}

__device__ __forceinline__ float pair_max_bf16(uint32_t pm) {  // the larger half of a packed bf16 pair, as fp32
    return fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xFFFF0000u));
}

// One chunk of a streaming lane: four 16-byte vectors of a tile (32 bf16 or 16 fp32 logits).  The chunk maximum goes
// to *cmax_slot for the second stage (2 bytes: the bf16 value, or the fp32 maximum rounded up to bf16).
template <bool BF16, bool GUARD>
__device__ __forceinline__ void process_chunk(const uint4* __restrict__ wb, int lane, int nvalid_vec, Acc& a,
                                              typename VT<BF16>::cm_t* cmax_slot) {
    using T = VT<BF16>;
    uint4 v[VEC_PER_LANE];
    uint32_t vm[VEC_PER_LANE];
#pragma unroll
    for (int i = 0; i < VEC_PER_LANE; ++i) {
        // A lane's chunk is 64 contiguous bytes (vectors 4 lane .. 4 lane + 3 of the warp's block), so that the second
        // stage re-reads a hit chunk as one 64-byte piece of one line instead of four sectors of four lines (random
        // DRAM accesses beside the stream cost it bandwidth).  The lanes take their four vectors in rotated order,
        // (i + lane / 2) mod 4, which spreads the eight lanes of a shared-memory phase over all bank groups.
        const int vi = 4 * lane + ((i + (lane >> 1)) & 3);
        if (!GUARD || vi < nvalid_vec)
            v[i] = wb[vi];
        else
            v[i] = make_uint4(T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD);
    }
    uint32_t cmk;
    if (BF16) {
#pragma unroll
        for (int i = 0; i < VEC_PER_LANE; ++i) vm[i] = hmax2_bf16(hmax2_bf16(v[i].x, v[i].y), hmax2_bf16(v[i].z, v[i].w));
        cmk = hmax2_bf16(hmax2_bf16(vm[0], vm[1]), hmax2_bf16(vm[2], vm[3]));
        a.rmax = hmax2_bf16(a.rmax, cmk);
        {
            // the larger half of the pair, as 16 bits: the halves swapped (one byte permute), one more packed maximum
            uint32_t sw;
            asm("prmt.b32 %0, %1, %1, 0x1032;" : "=r"(sw) : "r"(cmk));
            *cmax_slot = (typename T::cm_t)(hmax2_bf16(cmk, sw) & 0xFFFFu);
        }
        if (hmax2_bf16(cmk, a.thr) != a.thr) acc_raise<BF16>(a, pair_max_bf16(cmk));  // some half above the threshold
    } else {
        float m = -INFINITY;
#pragma unroll
        for (int i = 0; i < VEC_PER_LANE; ++i) {
            const float mi = fmaxf(fmaxf(__uint_as_float(v[i].x), __uint_as_float(v[i].y)),
                                   fmaxf(__uint_as_float(v[i].z), __uint_as_float(v[i].w)));
            vm[i] = __float_as_uint(mi);
            m = fmaxf(m, mi);
        }
        cmk = __float_as_uint(m);
        a.rmax = __float_as_uint(fmaxf(__uint_as_float(a.rmax), m));
        {
            // round toward +inf onto the bf16 grid: positive values round their magnitude up, negative ones truncate
            const uint32_t mb = cmk;
            *cmax_slot = (typename T::cm_t)((mb >> 31) ? (mb >> 16) : ((mb + 0xFFFFu) >> 16));
        }
        if (m > __uint_as_float(a.thr)) acc_raise<BF16>(a, m);
    }
#if GRAFT_VP_F32X2
    const uint64_t c2 = pack2(kLog2e, kLog2e), r2 = pack2(a.nref, a.nref);
#pragma unroll
    for (int i = 0; i < VEC_PER_LANE; ++i) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        if (BF16) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint64_t x2 = pack2(__uint_as_float(w[k] << 16), __uint_as_float(w[k] & 0xFFFF0000u));
                float t0, t1;
                unpack2(fma2(x2, c2, r2), t0, t1);
                const uint64_t e2 = pack2(ex2_approx(t0), ex2_approx(t1));
                if (k & 1)
                    a.a1 = add2(a.a1, e2);
                else
                    a.a0 = add2(a.a0, e2);
            }
        } else {
            float t0, t1, t2, t3;
            unpack2(fma2(pack2(__uint_as_float(w[0]), __uint_as_float(w[1])), c2, r2), t0, t1);
            unpack2(fma2(pack2(__uint_as_float(w[2]), __uint_as_float(w[3])), c2, r2), t2, t3);
            a.a0 = add2(a.a0, pack2(ex2_approx(t0), ex2_approx(t1)));
            a.a1 = add2(a.a1, pack2(ex2_approx(t2), ex2_approx(t3)));
        }
    }
#else
#pragma unroll
    for (int i = 0; i < VEC_PER_LANE; ++i) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        if (BF16) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xFFFF0000u);
                const float e0 = ex2_approx(fmaf(lo, kLog2e, a.nref)), e1 = ex2_approx(fmaf(hi, kLog2e, a.nref));
                if (k & 1) {
                    a.s2 += e0;
                    a.s3 += e1;
                } else {
                    a.s0 += e0;
                    a.s1 += e1;
                }
            }
        } else {
            a.s0 += ex2_approx(fmaf(__uint_as_float(w[0]), kLog2e, a.nref));
            a.s1 += ex2_approx(fmaf(__uint_as_float(w[1]), kLog2e, a.nref));
            a.s2 += ex2_approx(fmaf(__uint_as_float(w[2]), kLog2e, a.nref));
            a.s3 += ex2_approx(fmaf(__uint_as_float(w[3]), kLog2e, a.nref));
        }
    }
#endif
}

template <bool BF16>
__device__ __forceinline__ float acc_sum(const Acc& a) {
#if GRAFT_VP_F32X2
    float s0, s1, s2, s3;
    unpack2(a.a0, s0, s1);
    unpack2(a.a1, s2, s3);
    return (s0 + s1) + (s2 + s3);
#else
    return (a.s0 + a.s1) + (a.s2 + a.s3);
#endif
}

// (c, s) pairs stand for s * 2^c; merge two of them
__device__ __forceinline__ void merge_cs(float& c, float& s, float c2, float s2) {
    const float cn = fmaxf(c, c2);
    const float f1 = (c == -INFINITY) ? 0.f : ex2_approx(c - cn);
    const float f2 = (c2 == -INFINITY) ? 0.f : ex2_approx(c2 - cn);
    s = s * f1 + s2 * f2;
    c = cn;
}


// ---- shared-memory control block ---------------------------------------------------------------
struct __align__(16) EpiShared {  // private to one epilogue group
    uint64_t cand[kVpCandCap];
    uint64_t outk[kMaxK];
    uint32_t hits[kVpHitCap];
    uint16_t hthreads[NT];  // streaming threads whose maximum reaches T
    int nhits, ncand, nht, ovf;
    int tie_groups;  // groups of threads whose maximum is T (to 16 bits): many of them means bulk ties at T
    int fill_ninf;  // the threshold fell on -inf: the candidates are the finite elements plus the first -inf ones
    int fill_tie;   // too many chunks reach the threshold T (bulk ties at T): the candidates are the elements above T
                    // plus the first elements equal to T
    uint32_t Tv;
};
struct __align__(16) VpShared {
    EpiShared epi[kVpEpiGroups];
    uint32_t tmax[kVpBufs][NT];  // per-thread maxima of a finished segment, one buffer per segment in flight
    uint32_t gmax[kVpBufs][kVpGroups];  // the same maxima folded into 64 groups (lane, warp parity); zero when idle
    float wc[kVpBufs][NW], ws[kVpBufs][NW];
    volatile int abort_flag;
};

__device__ __forceinline__ void epi_bar(int group) { named_bar_sync(2 + group, kVpEpiThreads); }

// ---- epilogue-warp helpers (32 threads, warp-synchronous) ----------------------------------------------
// Append `key` for the lanes with pred set; returns the new count.  Entries beyond the capacity are dropped
// and *overflow is raised.
__device__ __forceinline__ int warp_append(uint64_t* buf, int n, int cap, bool pred, uint64_t key, int lane,
                                           int* overflow) {
    const uint32_t m = __ballot_sync(0xFFFFFFFFu, pred);
    if (pred) {
        const int pos = n + __popc(m & ((1u << lane) - 1u));
        if (pos < cap)
            buf[pos] = key;
        else
            *overflow = 1;
    }
    n += __popc(m);
    if (n > cap) {
        *overflow = 1;
        n = cap;
    }
    return n;
}

// Exact top-K of cand[0..n) by rank counting; result sorted descending in outk[0..min(n,K)).  Keys are
// distinct (ids are), so ranks are a permutation.
__device__ void warp_select_topk(EpiShared* sh, int n, int K, int lane) {
    __syncwarp();
    for (int i = lane; i < n; i += 32) {
        const uint64_t key = sh->cand[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (sh->cand[j] > key) ? 1 : 0;
        if (rank < K) sh->outk[rank] = key;
    }
    __syncwarp();
}

// The K-th largest chunk maximum of a segment (every streaming thread leaves one 16-bit maximum per tile), as a 16-bit
// order-preserving pattern; 0 when the segment has fewer than K chunks.  All 128 threads of an epilogue group; two
// histogram passes of eight bits each over the idle hit list.  Out of line: rows that need it are rare.
__device__ __noinline__ uint32_t epi_kth_chunk_max(EpiShared* es, const uint16_t* cmx, int max_tiles, int ntiles, int K,
                                                   int etid, int grp) {
    uint32_t* hist = es->hits;  // [0, 256) counts, [256] the bin found, [257] the count above it
    uint32_t prefix = 0u;
    int want = K;
#pragma unroll 1
    for (int pass = 0; pass < 2; ++pass) {
        for (int i = etid; i < 258; i += kVpEpiThreads) hist[i] = 0u;
        epi_bar(grp);
#pragma unroll 1
        for (int t = etid; t < NT; t += kVpEpiThreads) {
            const uint16_t* row = cmx + (size_t)t * max_tiles;
#pragma unroll 1
            for (int tile = 0; tile < ntiles; ++tile) {
                const uint32_t v = ord_from_bits((uint32_t)row[tile] << 16) >> 16;
                if (pass == 0)
                    atomicAdd(&hist[v >> 8], 1u);
                else if ((v >> 8) == prefix)
                    atomicAdd(&hist[v & 255u], 1u);
            }
        }
        epi_bar(grp);
        if (etid < 32) {  // the bin in which the count from the top reaches `want`: eight bins a lane
            uint32_t own = 0u;
#pragma unroll
            for (int i = 0; i < 8; ++i) own += hist[8 * etid + i];
            uint32_t above = own;  // inclusive sum over the lanes from this one up
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t o = __shfl_down_sync(0xFFFFFFFFu, above, d);
                if (etid + d < 32) above += o;
            }
            if (above >= (uint32_t)want && above - own < (uint32_t)want) {  // (one lane at most)
                uint32_t acc = above - own;
                for (int i = 7; i >= 0; --i) {
                    const uint32_t c = hist[8 * etid + i];
                    if (acc + c >= (uint32_t)want) {
                        hist[256] = (uint32_t)(8 * etid + i) | 0x100u;
                        hist[257] = acc;
                        break;
                    }
                    acc += c;
                }
            }
        }
        epi_bar(grp);
        const uint32_t bin = hist[256];
        if (bin == 0u) {  // fewer than K chunks (uniform)
            prefix = 0u;
            pass = 2;
        } else {
            prefix = (prefix << 8) | (bin & 255u);
            want -= (int)hist[257];
        }
        epi_bar(grp);  // (read before the next pass clears it)
    }
    return prefix;
}

// Exact top-K of cand[0..n) for hundreds of keys, K < n: ranking them against each other costs n^2 compares; here the
// K-th largest key is found by a search over its bits, two at a time with three counts each -- over the value word
// first; over the id word, among the keys of that value, only if more keys share the K-th largest value than are
// wanted -- and the K keys that reach it (keys are distinct: exactly K) are ranked into outk.  Whatever the keys'
// order or values.  All 128 threads of an epilogue group; the counts of its warps meet in the idle hit list.  Out of
// line: rows that need it are rare.
__device__ __noinline__ void epi_select_many(EpiShared* es, int n, int K, int etid, int grp) {
    uint32_t* cnt = es->hits;                       // [2 * 16 * 3] counts of the steps, [96], [97] above / at the value, [98] kept
    uint64_t* kept = (uint64_t*)(es->hits + 128);   // [K] the keys that reach the K-th largest
    const uint32_t* word = (const uint32_t*)es->cand;  // key i: id word at 2 i, value word at 2 i + 1
    for (int i = etid; i < 99; i += kVpEpiThreads) cnt[i] = 0u;
    epi_bar(grp);
    uint32_t vk = 0u, ik = 0u;  // the K-th largest key's value word and id word
    int want = K;
#pragma unroll 1
    for (int phase = 0; phase < 2; ++phase) {
        uint32_t kth = 0u;
#pragma unroll 1
        for (int step = 0; step < 16; ++step) {
            const int bit = 30 - 2 * step;
            const uint32_t t1 = kth | (1u << bit), t2 = kth | (2u << bit), t3 = kth | (3u << bit);
            int c1 = 0, c2 = 0, c3 = 0;
#pragma unroll 2
            for (int i = etid; i < n; i += kVpEpiThreads) {
                const uint32_t hi = word[2 * i + 1];
                const uint32_t x = phase == 0 ? hi : (hi == vk ? word[2 * i] : 0u);  // (an id word is never 0)
                c1 += (x >= t1) ? 1 : 0;
                c2 += (x >= t2) ? 1 : 0;
                c3 += (x >= t3) ? 1 : 0;
            }
            c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
            c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
            c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
            uint32_t* slot = cnt + (phase * 16 + step) * 3;
            if ((etid & 31) == 0) {
                atomicAdd(&slot[0], (uint32_t)c1);
                atomicAdd(&slot[1], (uint32_t)c2);
                atomicAdd(&slot[2], (uint32_t)c3);
            }
            epi_bar(grp);
            const int n1 = (int)slot[0], n2 = (int)slot[1], n3 = (int)slot[2];
            kth = n3 >= want ? t3 : (n2 >= want ? t2 : (n1 >= want ? t1 : kth));
        }
        if (phase == 1) {
            ik = kth;
            break;
        }
        vk = kth;
        int above = 0, at = 0;
        for (int i = etid; i < n; i += kVpEpiThreads) {
            const uint32_t hi = word[2 * i + 1];
            above += (hi > vk) ? 1 : 0;
            at += (hi == vk) ? 1 : 0;
        }
        above = __reduce_add_sync(0xFFFFFFFFu, above);
        at = __reduce_add_sync(0xFFFFFFFFu, at);
        if ((etid & 31) == 0) {
            atomicAdd(&cnt[96], (uint32_t)above);
            atomicAdd(&cnt[97], (uint32_t)at);
        }
        epi_bar(grp);
        want = K - (int)cnt[96];
        if ((int)cnt[97] == want) break;  // (uniform) every key of that value is wanted: ik = 0 lets them all through
    }
    const uint64_t kth_key = ((uint64_t)vk << 32) | ik;
    for (int i = etid; i < n; i += kVpEpiThreads) {
        const uint64_t k = es->cand[i];
        if (k >= kth_key) {
            const uint32_t pos = atomicAdd(&cnt[98], 1u);
            if (pos < (uint32_t)kMaxK) kept[pos] = k;
        }
    }
    epi_bar(grp);
    const int m = (int)cnt[98] < K ? (int)cnt[98] : K;
    if (etid < m) {
        const uint64_t k = kept[etid];
        int rank = 0;
        for (int j2 = 0; j2 < m; ++j2) rank += (kept[j2] > k) ? 1 : 0;
        es->outk[rank] = k;
    }
}

// ord() of the largest element of a 16-byte vector
template <bool BF16>
__device__ __forceinline__ uint32_t vec_max_ord(const uint4& x) {
    if (BF16) return ord_from_float(pair_max_bf16(hmax2_bf16(hmax2_bf16(x.x, x.y), hmax2_bf16(x.z, x.w))));
    return ord_from_float(fmaxf(fmaxf(__uint_as_float(x.x), __uint_as_float(x.y)),
                                fmaxf(__uint_as_float(x.z), __uint_as_float(x.w))));
}

// Exact selection over a whole segment straight from global memory.  Used only when the fast path's buffers
// overflowed, which means that most of the segment ties with its K-th largest element (rows that are flat, masked
// to -inf, or all but one element equal).  The running K-th best key is the filter: an element enters the buffer
// only if its key (value, then smaller id) beats it, and once the first K of a flat row are in, nothing else does.
// The segment's 16-byte aligned body is read in batches of one streaming warp's 2 KiB of a tile; a batch whose
// chunk maxima (left by the streaming warps) rule out a key above the filter is not read at all; the few elements
// before and after the body go one by one.
// When the buffer fills up, the best K are kept and the filter rises.
template <bool BF16>
__device__ int warp_fallback_select(EpiShared* sh, const VpParams& p, const Seg& sg,
                                    const typename VT<BF16>::cm_t* cmx, int lane, uint64_t thr) {
    using T = VT<BF16>;
    const int K = p.K;
    const char* rowp = p.logits + (size_t)sg.row * p.V * T::ESZ;
    // thr: keys must beat this one (on entry: what the threshold T of the fast path rules out, or 0)
    int n = 0, ovf = 0;
    // ranking n keys against each other costs n^2 / 32 steps per lane: the buffer is cut back to its best K well
    // before it is full (96 more keys at a time)
    constexpr int kFallbackFill = 128 - 32;
    auto shrink = [&]() {  // keep the best K of the buffer
        if (n > K) {
            warp_select_topk(sh, n, K, lane);
            if (lane < K) sh->cand[lane] = sh->outk[lane];
            thr = sh->outk[K - 1];
            n = K;
            __syncwarp();
        }
    };
    auto one_by_one = [&](int e_begin, int e_end) {
        for (int e0 = e_begin; e0 < e_end; e0 += 32) {
            const int e = e0 + lane;
            uint64_t key = 0;
            if (e < e_end) key = make_key(__float_as_uint(load_elem_f32(rowp + (size_t)e * T::ESZ, BF16)), (uint32_t)e);
            n = warp_append(sh->cand, n, kVpCandCap, e < e_end && key > thr, key, lane, &ovf);
            if (n > kFallbackFill) shrink();
        }
    };
    one_by_one(sg.e0, sg.e_body0);
    constexpr int U = 4;
    const int nvec = (int)(sg.body_bytes / 16);
    const uint4* body = (const uint4*)sg.body;
    for (int v0 = 0; v0 < nvec; v0 += 32 * U) {
        // The batch is one streaming warp's 2 KiB of a tile, and this lane's four consecutive vectors are the chunk whose
        // maximum (rounded up to bf16) that warp's lane left in cmx.  A chunk cannot hold a key above the filter if
        // its maximum is below the filter's value, or not above it while all its ids come after the filter's id.
        if (thr != 0ull) {
            const int tile = v0 / (TILE / 16), wb = (v0 % (TILE / 16)) / (32 * U);
            const uint32_t mx = ord_from_bits((uint32_t)cmx[(size_t)(wb * 32 + lane) * p.max_tiles + tile] << 16);
            const uint32_t v_thr = (uint32_t)(thr >> 32);
            const uint32_t first_id = (uint32_t)(sg.e_body0 + (v0 + 4 * lane) * T::EPV);
            const bool need = !(mx < v_thr || (mx <= v_thr && first_id > key_id(thr)));
            if (!__any_sync(0xFFFFFFFFu, need)) continue;  // (uniform)
        }
#pragma unroll 1
        for (int u = 0; u < U; ++u) {  // (one vector at a time: this path must not cost the kernel registers)
            const int v = v0 + u * 32 + lane;
            uint4 x = make_uint4(T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD);
            if (v < nvec) x = body[v];
            const uint32_t wv[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < T::EPV; ++q) {
                uint32_t xb;
                if (BF16)
                    xb = (q & 1) ? (wv[q >> 1] & 0xFFFF0000u) : (wv[q >> 1] << 16);
                else
                    xb = wv[q];
                const uint64_t key = v < nvec ? make_key(xb, (uint32_t)(sg.e_body0 + v * T::EPV + q)) : 0ull;
                n = warp_append(sh->cand, n, kVpCandCap, key > thr, key, lane, &ovf);
                if (n > kFallbackFill) shrink();  // (uniform)
            }
        }
    }
    one_by_one(sg.e_tail0, sg.e1);
    warp_select_topk(sh, n, K, lane);
    return n < K ? n : K;
}

// The outputs of a finished row from its pieces: C, S with sum_v 2^(z_v c) = S 2^C (c = fp32(log2 e)), the largest
// logit, and the K best keys.  One warp.  `internal`: a bounded wait ran out in a CTA that worked on this row.
__device__ __forceinline__ void vp_finalize(double Cd, double Sd, uint32_t Vm, int nk, int K, const uint64_t* keys,
                                            int lane, int32_t* topk_id, float* topk_lp, float* lse,
                                            int32_t* row_status, bool internal) {
    // The stream accumulates 2^(z c - ref) with c = fp32(log2 e), so (C + log2 S) ln 2 is the
    // log-sum-exp of the logits scaled by a = c ln 2 = 1 + 1.3e-8.  To first order that adds
    // (a - 1) E_q[z]; the largest logit stands in for the mean under q (the difference is a few
    // units times 1e-8).
    // every lane must use the same bits: the folds that produced C and S are butterflies of fused multiply-adds,
    // which leave the lanes an ulp apart, and log-probabilities of equal logits (and their order) must not depend on
    // the lane that writes them
    Cd = __shfl_sync(0xFFFFFFFFu, Cd, 0);
    Sd = __shfl_sync(0xFFFFFFFFu, Sd, 0);
    Vm = __shfl_sync(0xFFFFFFFFu, Vm, 0);
    const float vmax = __uint_as_float(bits_from_ord(Vm));
    const double a_minus_1 = (double)kLog2e * kLn2 - 1.0;
    const double lse_d = (Cd + log2(Sd)) * kLn2 - a_minus_1 * (double)vmax;
    const bool bad = !(Sd > 0.0) || !(Sd < 1e300) || Vm == 0u || vmax == INFINITY || vmax == -INFINITY || nk < K;
    if (lane < K) {
        const uint64_t key = lane < nk ? keys[lane] : 0ull;
        topk_id[lane] = lane < nk ? (int32_t)key_id(key) : -1;
        topk_lp[lane] = lane < nk ? (float)((double)key_value(key) - lse_d) : 0.f;
    }
    if (lane == 0) {
        *lse = (float)lse_d;
        *row_status = (bad ? GRAFT_ST_BAD_LOGITS : 0) | (internal ? GRAFT_ST_INTERNAL : 0);
    }
}

template <bool BF16>
__global__ void __launch_bounds__(kVpThreads, 1) vocab_pass_kernel(const VpParams p) {
    using T = VT<BF16>;
    using cm_t = typename T::cm_t;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    pdl_launch_dependents();  // the edge-score kernel's CTAs may move in as this grid's CTAs leave; they wait for it
    unsigned char* ring = smem_raw;
    uint64_t* bars = (uint64_t*)(ring + (size_t)p.stages * TILE);  // full[8], empty[8], ready[4], done[4]
    VpShared* sh = (VpShared*)(bars + 24);
    cm_t* cmax = (cm_t*)(sh + 1);  // [kVpBufs][n_cmax]

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long G = gridDim.x;
    const long long q0 = cta_start(blockIdx.x, p.Q, G), q1 = cta_start(blockIdx.x + 1, p.Q, G);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 8);
    const uint32_t ready0 = smem_u32(bars + 16), done0 = smem_u32(bars + 20);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, NW);
        }
        for (int s = 0; s < kVpBufs; ++s) {
            mbar_init(ready0 + 8 * s, NW);
            mbar_init(done0 + 8 * s, 1);
        }
        mbar_fence_init();
        sh->abort_flag = 0;
    }
    if (tid < kVpBufs * kVpGroups) (&sh->gmax[0][0])[tid] = 0u;
    __syncthreads();
    // Launched with programmatic stream serialization inside a round: the CTA is set up while the kernel ahead of it in
    // the stream (the previous round's walk or tree kernel) drains; nothing is read or written before that kernel has
    // completed (the logits may come from it, and the scratch this kernel writes is read by the previous round's
    // kernels).  Launched the ordinary way this returns at once.
    pdl_wait();

    if (warp == PROD_WARP) {
        // ------------------------------ producer warp --------------------------------------------
        if (lane == 0) {
            uint64_t policy = 0;
            if (p.use_hint) policy = l2_policy_evict_first();
            uint32_t t = 0, st = 0, ph = 1;  // ph: parity of the "empty" phase to wait for (first lap: none)
            const uint32_t nst = (uint32_t)p.stages;
            SegIter it = seg_iter_begin<BF16>(p, q0, q1);
            Seg sg;
            while (seg_iter_next<BF16>(p, it, sg)) {
                // the segment this CTA visits last is read the ordinary way instead of evict-first: the second
                // stage of its epilogue, which nothing overlaps any more, then finds its chunks in L2
                const bool hint = p.use_hint && !seg_iter_at_end(it);
                for (int tile = 0; tile < sg.ntiles; ++tile, ++t) {
                    if (t >= nst) mbar_wait_bounded_hint(empty0 + 8 * st, ph, &sh->abort_flag, kVpIdleHintNs);
#ifdef GRAFT_TEST_WITHHOLD_TILE
                    // Test builds only (the shipped library is never compiled with this): CTA 0 does not issue the
                    // copy of one of its tiles, so that the streaming warps' bounded wait for it runs out and the
                    // time-out path (error flag, status bit, drain) can be exercised without faulting anything.
                    if (blockIdx.x == 0 && t == GRAFT_TEST_WITHHOLD_TILE) {
                        if (++st == nst) {
                            st = 0;
                            ph ^= 1;
                        }
                        continue;
                    }
#endif
                    uint32_t off = (uint32_t)tile * TILE;
                    uint32_t bytes = sg.body_bytes - off < (uint32_t)TILE ? sg.body_bytes - off : (uint32_t)TILE;
                    mbar_arrive_expect_tx(full0 + 8 * st, bytes);
                    if (hint)
                        tma_load_1d_hint(smem_u32(ring + (size_t)st * TILE), sg.body + off, bytes, full0 + 8 * st, policy);
                    else
                        tma_load_1d(smem_u32(ring + (size_t)st * TILE), sg.body + off, bytes, full0 + 8 * st);
                    if (++st == nst) {
                        st = 0;
                        ph ^= 1;
                    }
                }
            }
            if (sh->abort_flag) {
                // a consumer gave up: make sure none of our copies is still in flight before the CTA retires
                for (uint32_t back = 0; back < nst && back < t; ++back) {
                    const uint32_t tt = t - 1 - back;
                    uint32_t tries = 0;
                    while (!mbar_try_wait(full0 + 8 * (tt % nst), (tt / nst) & 1) && ++tries < GRAFT_SPIN_LIMIT) {
                    }
                }
            }
        }
    } else if (warp < NW) {
        // ------------------------------ streaming warps ------------------------------------------
        uint32_t st = 0, ph = 0;  // ring position and parity of the "full" phase to wait for
        const uint32_t nst = (uint32_t)p.stages;
        uint32_t k = 0;           // segment counter: hand-over buffers are indexed by k % kVpBufs
        SegIter it = seg_iter_begin<BF16>(p, q0, q1);
        Seg sg;
        for (; seg_iter_next<BF16>(p, it, sg); ++k) {
            const uint32_t pb = k % kVpBufs;
            Acc a;
            acc_init<BF16>(a);
            // buffer pb is free once the epilogue of segment k - kVpBufs is done
            if (k >= kVpBufs) mbar_wait_bounded(done0 + 8 * pb, ((k / kVpBufs) - 1u) & 1u, &sh->abort_flag);
            {
                const int nfull = (int)(sg.body_bytes / TILE);
                cm_t* slot = cmax + (size_t)pb * p.n_cmax + (size_t)tid * p.max_tiles;  // this thread's slots, by tile
                for (int tile = 0; tile < sg.ntiles; ++tile, ++slot) {
                    mbar_wait_bounded_hint(full0 + 8 * st, ph, &sh->abort_flag, 2000u);
                    const uint4* wb = (const uint4*)(ring + (size_t)st * TILE + (size_t)warp * WBLK);
                    if (tile < nfull) {
                        process_chunk<BF16, false>(wb, lane, 0, a, slot);
                    } else {
                        int nv = ((int)(sg.body_bytes - (uint32_t)tile * TILE) - warp * WBLK) / 16;
                        nv = nv < 0 ? 0 : (nv > WBLK / 16 ? WBLK / 16 : nv);
                        process_chunk<BF16, true>(wb, lane, nv, a, slot);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(empty0 + 8 * st);
                    if (++st == nst) {
                        st = 0;
                        ph ^= 1;
                    }
                }
            }
            // hand the segment over to the epilogue warp
            // (a thread that saw no data keeps 0 = nothing seen)
            const uint32_t tmo = sg.ntiles > 0 ? ord_from_float(BF16 ? pair_max_bf16(a.rmax) : __uint_as_float(a.rmax)) : 0u;
            sh->tmax[pb][tid] = tmo;
            atomicMax(&sh->gmax[pb][(warp & 1) * 32 + lane], tmo);
            {
                // the warp's piece of the log-sum-exp: the largest reference of its lanes (one integer reduction over
                // the order-preserving images), every lane's sum rescaled to it once, then a butterfly of plain adds
                // (a fixed order: the result does not depend on timing)
                const uint32_t co = __reduce_max_sync(0xFFFFFFFFu, ord_from_float(a.ref));
                const float c = __uint_as_float(bits_from_ord(co));
                float s = (a.ref == -INFINITY) ? 0.f : acc_sum<BF16>(a) * ex2_approx(a.ref - c);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
                if (lane == 0) {
                    sh->wc[pb][warp] = c;
                    sh->ws[pb][warp] = s;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(ready0 + 8 * pb);
        }
    } else if (warp == COS_WARP) {
        // ------------------------------ cosine warp ----------------------------------------------
        // Adjacent-position cosines of the SABA state (Eq. 15): a few pairs of hidden-state rows per CTA, read
        // beside the logits stream (under 3 % of its bytes) so that nothing downstream waits for them.
        if (p.cos_out != nullptr) {
            const int npairs = (p.rows / p.L) * (p.L - 1);
            for (int q = (int)blockIdx.x; q < npairs; q += (int)gridDim.x) {
                const int sb = q / (p.L - 1), d = q - sb * (p.L - 1);
                const double r = warp_adjacent_cosine(p.hidden, p.hidden_bf16, p.hidden_dim,
                                                      ((size_t)sb * p.L + d) * p.hidden_dim, lane);
                if (lane == 0) p.cos_out[(size_t)sb * p.L + d] = r;
            }
        }
    } else {
        // ------------------------------ epilogue groups (four warps each) ------------------------
        // Group g finishes the segments with k % 2 == g, so a group has two segment times for one epilogue.
        // Warp 0 of a group owns the hand-over barriers and the sequential parts; the data-parallel parts (which
        // chunks reach T, re-reading them, ranking the candidates) are shared by the group's 128 threads.
        const int grp = (warp - NW) / (kVpEpiThreads / 32), ew = (warp - NW) % (kVpEpiThreads / 32);
        const int etid = (tid - NT) % kVpEpiThreads;
        EpiShared* const es = &sh->epi[grp];
        uint32_t k = 0;
        SegIter it = seg_iter_begin<BF16>(p, q0, q1);
        Seg sg;
        for (; seg_iter_next<BF16>(p, it, sg); ++k) {
            if ((int)(k % kVpEpiGroups) != grp) continue;
            const uint32_t pb = k % kVpBufs;
            const char* rowp = p.logits + (size_t)sg.row * p.V * T::ESZ;
            const cm_t* cmx = cmax + (size_t)pb * p.n_cmax;
            if (ew == 0) mbar_wait_bounded_hint(ready0 + 8 * pb, (k / kVpBufs) & 1u, &sh->abort_flag, kVpIdleHintNs);
            float c = -INFINITY, s = 0.f;
            uint32_t vmo = 0;
            if (ew == 0) {
                int overflow = 0, ncand = 0;
                // (a) log-sum-exp pieces of the streaming warps
                c = lane < NW ? sh->wc[pb][lane] : -INFINITY;
                s = lane < NW ? sh->ws[pb][lane] : 0.f;
                // (b) ragged head / tail that the 16-byte bulk copies cannot carry: plain loads, every element a
                //     candidate (at most 7 + 7 elements unless the whole segment is shorter than 16 bytes)
                {
                    const int nhead = sg.e_body0 - sg.e0, ntail = sg.e1 - sg.e_tail0;
                    for (int i0 = 0; i0 < nhead + ntail; i0 += 32) {
                        const int i = i0 + lane;
                        const bool in = i < nhead + ntail;
                        uint64_t key = 0;
                        if (in) {
                            const int e = i < nhead ? sg.e0 + i : sg.e_tail0 + (i - nhead);
                            const float x = load_elem_f32(rowp + (size_t)e * T::ESZ, BF16);
                            const uint32_t o = ord_from_float(x);
                            vmo = o > vmo ? o : vmo;
                            // x log2(e) = c1 + r with c1 the rounded product and r its exact remainder (one FMA):
                            // 2^r = 1 + r ln 2 keeps what the rounding of c1 drops (up to 2e-6 of the term at
                            // |x| = 30, which is the whole error of the row when its largest logit sits here)
                            float c1 = __fmul_rn(x, kLog2e);
                            float s1 = fmaf(fmaf(x, kLog2e, -c1), 0.69314718f, 1.0f);
                            if (x == -INFINITY) {
                                c1 = -INFINITY;
                                s1 = 0.f;
                            } else if (!(x < INFINITY)) {
                                s1 = NAN;  // +inf or NaN poisons the sum and marks the row
                                c1 = 0.f;
                            }
                            merge_cs(c, s, c1, s1);
                            key = make_key(__float_as_uint(x), (uint32_t)e);
                        }
                        ncand = warp_append(es->cand, ncand, kVpCandCap, in, key, lane, &overflow);
                    }
                }
                // (c) T = the K-th largest group maximum, truncated to its top 16 bits: a lower bound of
                //     the K-th largest element of the segment's body (0 when fewer than K threads saw data)
                uint32_t Tv = 0;
                int tie_groups = 0;
                {
                    // over 64 group maxima rather than the 512 thread maxima: any partition of the elements into
                    // at least K groups gives a lower bound, and this one costs an eighth of the compares for about
                    // a third more candidates (groups = (lane, warp parity), so that a segment that only reaches
                    // two streaming warps still fills all of them)
                    uint32_t mine[kVpGroups / 32];
#pragma unroll
                    for (int i = 0; i < kVpGroups / 32; ++i) {
                        mine[i] = sh->gmax[pb][i * 32 + lane];
                        sh->gmax[pb][i * 32 + lane] = 0u;  // idle again (published by the `done` arrival below)
                        vmo = mine[i] > vmo ? mine[i] : vmo;
                    }
                    for (int bit = 30; bit >= 16; bit -= 2) {  // two bits per step: three independent counts
                        const uint32_t t1 = Tv | (1u << bit), t2 = Tv | (2u << bit), t3 = Tv | (3u << bit);
                        int c1 = 0, c2 = 0, c3 = 0;
#pragma unroll
                        for (int i = 0; i < kVpGroups / 32; ++i) {
                            c1 += (mine[i] >= t1) ? 1 : 0;
                            c2 += (mine[i] >= t2) ? 1 : 0;
                            c3 += (mine[i] >= t3) ? 1 : 0;
                        }
                        c1 = __reduce_add_sync(0xFFFFFFFFu, c1);
                        c2 = __reduce_add_sync(0xFFFFFFFFu, c2);
                        c3 = __reduce_add_sync(0xFFFFFFFFu, c3);
                        Tv = c3 >= p.K ? t3 : (c2 >= p.K ? t2 : (c1 >= p.K ? t1 : Tv));
                    }
#pragma unroll
                    for (int i = 0; i < kVpGroups / 32; ++i) tie_groups += ((mine[i] ^ Tv) >> 16) == 0u ? 1 : 0;
                    tie_groups = __reduce_add_sync(0xFFFFFFFFu, tie_groups);
                }
                // fold (c, s, max) across the warp
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    const float c2 = __shfl_xor_sync(0xFFFFFFFFu, c, d);
                    const float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, d);
                    merge_cs(c, s, c2, s2);
                }
                vmo = __reduce_max_sync(0xFFFFFFFFu, vmo);
                overflow = __any_sync(0xFFFFFFFFu, overflow);
                // A threshold at -inf (a vocabulary masked down to fewer finite tokens than the filter needs) would let
                // every element through.  The K best are then the finite elements and, after them, the -inf elements
                // of smallest id: the filter rises to the lowest finite value and the first K -inf elements of the
                // segment are added below.
                const bool ninf = Tv <= kOrdNegInf;
                if (ninf) Tv = kOrdNegInf + 1u;
                if (lane == 0) {
                    es->fill_ninf = ninf ? 1 : 0;
                    es->fill_tie = 0;
                    es->Tv = Tv;
                    es->nhits = 0;
                    es->nht = 0;
                    es->ncand = ncand;
                    es->ovf = overflow;
                    es->tie_groups = tie_groups;
                }
            }
            epi_bar(grp);
            uint32_t Tv = es->Tv;
            // (d) chunks whose stored maximum reaches T: only threads whose own maximum reaches T can have one.
            //     List positions come from shared-memory atomics (the order does not matter: the final selection
            //     ranks exact keys).  A hit is recorded as the byte offset of the chunk's first vector.
            for (int t = etid; t < NT; t += kVpEpiThreads) {
                const uint32_t x = sh->tmax[pb][t];
                if (x >= Tv && x != 0u) es->hthreads[atomicAdd(&es->nht, 1)] = (uint16_t)t;
            }
            epi_bar(grp);
            // Te: what a chunk's maximum (and, below, an element) must reach.  T itself at first.  If more chunks reach T
            // than the list holds, either thousands of elements tie with T (a flat rest under a few winners: most of the
            // 64 group maxima are T itself) or T is a poor bound (the groups of threads are a partition that a pattern in
            // step with the lanes defeats: a row of ramps as long as a warp's block leaves half the groups' maxima far down
            // every ramp).  Ties: the scan is repeated for what lies above T, and the first elements equal to T in id
            // order are taken by a walk over the chunks further down.  A poor bound: T is raised to the K-th largest chunk
            // maximum, the best bound the chunk maxima give, and the scan is repeated.  Whichever comes first, the other
            // follows if the list overflows again: four scans at most, then the exact selection.
            uint32_t Te = Tv;
            bool refined = false, tied = false;
            for (int pass = 0;; ++pass) {  // (uniform)
                // (listed thread, tile) pairs, four per thread at a time with their loads in flight together; the pair's
                // thread comes from a multiplication (idx / ntiles for idx < 2^16 and ntiles < 2^16, exactly)
                const int npairs = es->nht * sg.ntiles;
                const uint32_t magic = sg.ntiles > 1 ? 0xFFFFFFFFu / (uint32_t)sg.ntiles + 1u : 0u;  // ceil(2^32 / ntiles)
                constexpr int PU = 4;
                bool stop = false;
                for (int base = 0; base < npairs && !stop; base += kVpEpiThreads * PU) {
                    uint32_t raw[PU], off[PU];
#pragma unroll
                    for (int u = 0; u < PU; ++u) {
                        const int idx = base + u * kVpEpiThreads + etid;
                        raw[u] = 0u;
                        off[u] = 0u;
                        if (idx < npairs) {
                            const int h = sg.ntiles > 1 ? (int)__umulhi((uint32_t)idx, magic) : idx, tile = idx - h * sg.ntiles;
                            const uint32_t t = es->hthreads[h];
                            raw[u] = cmx[(size_t)t * p.max_tiles + tile];
                            off[u] = (uint32_t)tile * TILE + (t >> 5) * WBLK + (t & 31) * 64;
                        }
                    }
#pragma unroll
                    for (int u = 0; u < PU; ++u) {
                        if (ord_from_bits(raw[u] << 16) >= Te && base + u * kVpEpiThreads + etid < npairs && !stop) {
                            const int pos = atomicAdd(&es->nhits, 1);
                            if (pos >= kVpHitCap)
                                stop = true;  // too many: the exact selection over the segment takes over
                            else
                                es->hits[pos] = off[u];
                        }
                    }
                }
                epi_bar(grp);
                // (a list several times as long as a good bound leaves it -- about K chunks -- also says that T is poor:
                // its chunks would overflow the key buffer)
                const bool over = es->nhits > kVpHitCap;
                if (es->fill_ninf || (refined && tied)) break;  // (uniform)
                if (!over && !(pass == 0 && es->nhits > 5 * p.K && es->tie_groups < 16)) break;  // (uniform)
                epi_bar(grp);  // (everybody has read the count)
                if (!refined && (tied || !BF16 || es->tie_groups < 16)) {
                    uint32_t kth = epi_kth_chunk_max(es, cmx, p.max_tiles, sg.ntiles, p.K, etid, grp);
                    // (fp32 logits: the stored maxima are rounded up to bf16, the pattern below is a bound)
                    if (!BF16 && kth > 0u) kth -= 1u;
                    refined = true;
                    if ((kth << 16) > Tv || !over) {  // (uniform; the search used the hit list: scan again in any case)
                        if ((kth << 16) > Tv) Tv = kth << 16;
                        Te = Tv;
                        tied = false;
                        if (etid == 0) {
                            es->nhits = 0;
                            es->fill_tie = 0;
                            es->Tv = Tv;
                        }
                        epi_bar(grp);
                        continue;
                    }
                    if (tied) break;  // (no better bound and what lies above T overflows the list: the exact selection)
                }
                if (!BF16 || tied) break;
                tied = true;
                if (etid == 0) {
                    es->nhits = 0;
                    es->fill_tie = 1;
                }
                Te = Tv + 0x10000u;  // (the next bf16 value up, whatever the sign: T holds the value's upper 16 bits)
                epi_bar(grp);
            }
            // (e) the 16-byte vectors of the hit chunks, re-read from global memory; elements >= T become keys.
            //     A thread issues its loads of a round before it uses any: under a saturated memory system one
            //     round trip costs microseconds.
            {
                // (with too many hits nothing is re-read: a segment that is mostly ties would send every element
                // through one shared counter)
                const bool hit_ovf = es->nhits > kVpHitCap;
                const int nhits = hit_ovf ? 0 : es->nhits;
                if (etid == 0 && hit_ovf) es->ovf = 1;
                constexpr int RU = 2;
                const int nvec = nhits * VEC_PER_LANE;
                bool full = false;
                for (int base = 0; base < nvec && !full; base += kVpEpiThreads * RU) {
                    uint4 vv[RU];
                    uint32_t offs[RU];
#pragma unroll
                    for (int u = 0; u < RU; ++u) {
                        const int i = base + u * kVpEpiThreads + etid;
                        vv[u] = make_uint4(T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD);
                        offs[u] = 0xFFFFFFFFu;
                        if (i < nvec) {
                            const uint32_t off = es->hits[i / VEC_PER_LANE] + (uint32_t)(i % VEC_PER_LANE) * 16u;
                            if (off < sg.body_bytes) {
                                offs[u] = off;
                                vv[u] = *(const uint4*)(sg.body + off);
                            }
                        }
                    }
#pragma unroll
                    for (int u = 0; u < RU; ++u) {
                        if (offs[u] == 0xFFFFFFFFu) continue;
                        // (three of a hit chunk's four vectors hold nothing that reaches T: one test for the vector)
                        if (vec_max_ord<BF16>(vv[u]) < Te) continue;
                        const uint32_t wv[4] = {vv[u].x, vv[u].y, vv[u].z, vv[u].w};
#pragma unroll
                        for (int j = 0; j < T::EPV; ++j) {
                            uint32_t xb;
                            if (BF16)
                                xb = (j & 1) ? (wv[j >> 1] & 0xFFFF0000u) : (wv[j >> 1] << 16);
                            else
                                xb = wv[j];
                            if (ord_from_bits(xb) >= Te && !full) {
                                const int pos = atomicAdd(&es->ncand, 1);
                                if (pos < kVpCandCap)
                                    es->cand[pos] = make_key(xb, (uint32_t)(sg.e_body0 + offs[u] / T::ESZ + j));
                                else
                                    full = true;  // (the count stays above the capacity: the exact selection takes over)
                            }
                        }
                    }
                }
            }
            epi_bar(grp);
            if (es->fill_ninf || es->fill_tie) {  // (uniform)
                if (ew == 0) {
                    // The first K elements equal to -inf (or, for bulk ties, to T) of the segment's body in id order (the
                    // few elements before and after the body are candidates already): a walk over the chunks in id
                    // order -- tile, streaming warp, lane -- that reads only chunks whose stored maximum reaches T (any
                    // chunk when the value looked for is -inf), 32 elements at a time.  Every chunk read for ties holds
                    // one at least unless a larger element put it on the list, so the walk is short wherever the ties
                    // are; the walk for -inf gives up after 256 chunks and the exact selection takes over.
                    const bool tie = es->fill_tie != 0;
                    const uint32_t T16 = Tv >> 16;
                    // (K chunks or more with an element above T: no tied element is wanted.  Otherwise fewer than 2 K
                    // visits find K tied elements or the end of the segment.)
                    int need = tie && es->nhits >= p.K ? 0 : p.K, visits = 0;
                    const int max_visits = tie ? 2 * p.K : 256;
                    bool gave_up = false;
                    for (int blk = 0; blk < sg.ntiles * NW && need > 0; ++blk) {
                        const int tile = blk / NW, w = blk % NW;
                        const uint32_t cm = ord_from_bits((uint32_t)cmx[(size_t)(w * 32 + lane) * p.max_tiles + tile] << 16) >> 16;
                        uint32_t todo = __ballot_sync(0xFFFFFFFFu, !tie || cm >= T16);
                        while (todo != 0u && need > 0) {  // (uniform)
                            if (++visits > max_visits) {
                                gave_up = true;
                                need = 0;
                                break;
                            }
                            const uint32_t off = (uint32_t)tile * TILE + (uint32_t)w * WBLK + (uint32_t)(__ffs(todo) - 1) * 64u +
                                                 (uint32_t)lane * T::ESZ;
                            todo &= todo - 1u;
                            uint32_t xb = 0u;
                            bool is = false;
                            if (lane < 64 / T::ESZ && off < sg.body_bytes) {
                                xb = __float_as_uint(load_elem_f32(sg.body + off, BF16));
                                is = tie ? (ord_from_bits(xb) >> 16) == T16 : xb == 0xFF800000u;  // (-0 and +0 are one value)
                            }
                            const uint32_t mk = __ballot_sync(0xFFFFFFFFu, is);
                            if (is && __popc(mk & ((1u << lane) - 1u)) < need) {
                                const int pos = atomicAdd(&es->ncand, 1);
                                if (pos < kVpCandCap) es->cand[pos] = make_key(xb, (uint32_t)sg.e_body0 + off / T::ESZ);
                            }
                            need -= __popc(mk);
                        }
                    }
                    if (gave_up && lane == 0) es->ovf = 1;
                }
                epi_bar(grp);
            }
            // (f) exact top-K of the candidates by rank counting (keys are distinct, so ranks are a permutation)
            // (ranking n candidates costs n^2 compares shared by 128 threads: beyond 256 -- rows whose large elements sit
            // side by side, such as sorted rows, fill every chunk that reaches T with candidates -- one warp finds the
            // K-th largest key by its bits instead)
            const bool overflow = es->ovf != 0 || es->ncand > kVpRankCap;
            const int ncand = es->ncand < kVpCandCap ? es->ncand : kVpCandCap;
            int nk = ncand < p.K ? ncand : p.K;
            if (!overflow) {
                // two neighbouring lanes per candidate, each over every other key, two running counts each
                for (int i0 = 0; i0 < ncand; i0 += kVpEpiThreads / 2) {
                    const int i = i0 + (etid >> 1);
                    const uint64_t key = i < ncand ? es->cand[i] : ~0ull;
                    int r0 = 0, r1 = 0;
                    for (int j = etid & 1; j < ncand; j += 4) {
                        r0 += (es->cand[j] > key) ? 1 : 0;
                        r1 += (j + 2 < ncand && es->cand[j + 2] > key) ? 1 : 0;
                    }
                    int rank = r0 + r1;
                    rank += __shfl_xor_sync(0xFFFFFFFFu, rank, 1);
                    if (i < ncand && (etid & 1) == 0 && rank < p.K) es->outk[rank] = key;
                }
            } else if (es->ovf == 0 && es->ncand <= kVpCandCap) {  // (uniform; every candidate is in the buffer)
                epi_select_many(es, ncand, p.K, etid, grp);
            } else if (ew == 0) {
                // (T is a lower bound of the K-th largest element: the filter starts there, not at nothing -- a row sorted
                // in ascending order would otherwise send every element through the buffer; with the threshold moved up
                // from -inf, elements equal to -inf may be among the K best and nothing is ruled out)
                nk = warp_fallback_select<BF16>(es, p, sg, cmx, lane, es->fill_ninf ? 0ull : ((uint64_t)Tv << 32) - 1ull);
            }
            epi_bar(grp);
            if (ew != 0) continue;
            // the double-buffered arrays of parity pb may be reused from here on
            __syncwarp();
            if (lane == 0) mbar_arrive(done0 + 8 * pb);
            // (g) finish the row, or leave a record for the CTA that arrives last
            // (a whole row is nobody else's: the divisions that find a shared row's CTAs are for partial rows only)
            const bool whole_row = sg.e0 == 0 && sg.e1 == p.V;
            const long long x0 = (long long)sg.row * p.nq;
            const int c_first = whole_row ? (int)blockIdx.x : cta_of(x0, p.Q, G);
            const int c_last = whole_row ? (int)blockIdx.x : cta_of(x0 + p.nq - 1, p.Q, G);
            const int nseg = c_last - c_first + 1;
            double Cd = (double)c, Sd = (double)s;
            uint32_t Vm = vmo;
            bool finish = (nseg == 1);
            int rec_internal = 0;  // a bounded wait ran out in one of the CTAs that left a record for this row
            if (nseg > 1) {
                const int my_first_row = (int)(q0 / p.nq);
                VpRecord* rec = p.records + (size_t)blockIdx.x * 2 + (sg.row == my_first_row ? 0 : 1);
                if (lane < kMaxK) rec->keys[lane] = lane < nk ? es->outk[lane] : 0ull;
                if (lane == 0) {
                    rec->c = c;
                    rec->s = s;
                    rec->vmax = __uint_as_float(vmo);
                    rec->nkeys = (uint32_t)nk | (sh->abort_flag ? 0x80000000u : 0u);
                }
                __threadfence();
                __syncwarp();
                int old = 0;
                if (lane == 0) {
                    old = atomicAdd(p.row_counter + sg.row, 1);
                    __threadfence();
                }
                old = __shfl_sync(0xFFFFFFFFu, old, 0);
                if (old == nseg - 1) {
                    finish = true;
                    // merge the records of CTAs c_first..c_last, a round at a time
                    const int per_round = (kVpCandCap - kMaxK) / kMaxK;
                    int have = 0;
                    for (int c0 = c_first; c0 <= c_last; c0 += per_round) {
                        const int c1 = c0 + per_round - 1 < c_last ? c0 + per_round - 1 : c_last;
                        int n = have, ovf = 0;
                        for (int i0 = 0; i0 < (c1 - c0 + 1) * kMaxK; i0 += 32) {
                            const int i = i0 + lane;
                            const int cc = c0 + i / kMaxK, kk = i % kMaxK;
                            const int c_row0 = (int)(cta_start(cc, p.Q, G) / p.nq);
                            const VpRecord* r = p.records + (size_t)cc * 2 + (sg.row == c_row0 ? 0 : 1);
                            const uint64_t key = __ldcg((const unsigned long long*)&r->keys[kk]);
                            n = warp_append(es->cand, n, kVpCandCap, key != 0ull, key, lane, &ovf);
                        }
                        warp_select_topk(es, n, p.K, lane);
                        have = n < p.K ? n : p.K;
                        if (lane < have) es->cand[lane] = es->outk[lane];
                        __syncwarp();
                    }
                    nk = have;
                    // log-sum-exp pieces, folded in double
                    double Cm = -INFINITY;
                    uint32_t vm = 0;
                    for (int cc = c_first + lane; cc <= c_last; cc += 32) {
                        const int c_row0 = (int)(cta_start(cc, p.Q, G) / p.nq);
                        const VpRecord* r = p.records + (size_t)cc * 2 + (sg.row == c_row0 ? 0 : 1);
                        if (__ldcg(&r->nkeys) & 0x80000000u) rec_internal = 1;
                        const float rc = __ldcg(&r->c);
                        const uint32_t rv = __float_as_uint(__ldcg(&r->vmax));
                        Cm = fmax(Cm, (double)rc);
                        vm = vm > rv ? vm : rv;
                    }
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) {
                        Cm = fmax(Cm, __shfl_xor_sync(0xFFFFFFFFu, Cm, d));
                        const uint32_t v2 = __shfl_xor_sync(0xFFFFFFFFu, vm, d);
                        vm = vm > v2 ? vm : v2;
                    }
                    double S = 0.0;
                    for (int cc = c_first + lane; cc <= c_last; cc += 32) {
                        const int c_row0 = (int)(cta_start(cc, p.Q, G) / p.nq);
                        const VpRecord* r = p.records + (size_t)cc * 2 + (sg.row == c_row0 ? 0 : 1);
                        const float rc = __ldcg(&r->c), rs = __ldcg(&r->s);
                        if (rc != -INFINITY)
                            S += (double)rs * exp2((double)rc - Cm);
                        else if (rs != rs)
                            S += (double)rs;
                    }
#pragma unroll
                    for (int d = 16; d > 0; d >>= 1) S += __shfl_xor_sync(0xFFFFFFFFu, S, d);
                    rec_internal = __any_sync(0xFFFFFFFFu, rec_internal);
                    Cd = Cm;
                    Sd = S;
                    Vm = vm;
                    if (lane == 0) p.row_counter[sg.row] = 0;
                }
            }
            if (finish && p.partial_out != nullptr) {
                graft_vocab_partial* po = p.partial_out + sg.row;
                if (lane < kMaxK) po->keys[lane] = lane < nk ? es->outk[lane] : 0ull;
                if (lane == 0) {
                    po->c = Cd;
                    po->s = Sd;
                    po->vmax_ord = Vm;
                    po->nkeys = (uint32_t)nk | ((rec_internal || sh->abort_flag) ? 0x80000000u : 0u);
                }
            } else if (finish) {
                vp_finalize(Cd, Sd, Vm, nk, p.K, es->outk, lane, p.topk_id + (size_t)sg.row * p.K,
                            p.topk_lp + (size_t)sg.row * p.K, p.lse + sg.row, p.row_status + sg.row,
                            rec_internal || sh->abort_flag != 0);
            }
            __syncwarp();
        }
    }
    __syncthreads();
    if (tid == 0 && sh->abort_flag) atomicOr(p.errflag, 1);
}

// ---- vocabulary-parallel merge: one CTA of 128 threads per row ---------------------------------------------------
constexpr int kMergeMaxShards = 64;
struct MergeParams {
    const graft_vocab_partial* parts;  // [n_shards, rows]
    int n_shards, rows, K;
    int32_t v_offset[kMergeMaxShards];
    int32_t* topk_id;
    float* topk_lp;
    float* lse;
    int32_t* row_status;
};
__global__ void __launch_bounds__(128) vocab_merge_kernel(const MergeParams p) {
    __shared__ uint64_t cand[kMergeMaxShards * kMaxK];
    __shared__ uint64_t outk[kMaxK];
    __shared__ double sC[kMergeMaxShards], sS[kMergeMaxShards];
    __shared__ uint32_t sV[kMergeMaxShards], sN[kMergeMaxShards];
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31;
    const int n = p.n_shards * kMaxK;
    // the shards' keys with global token ids (an empty slot stays 0 and ranks below every key)
    for (int i = tid; i < n; i += 128) {
        const int sidx = i / kMaxK, kk = i % kMaxK;
        const graft_vocab_partial* r = p.parts + (size_t)sidx * p.rows + row;
        uint64_t key = kk < (int)(r->nkeys & 0x7FFFFFFFu) ? r->keys[kk] : 0ull;
        if (key != 0ull) key = make_key(bits_from_ord((uint32_t)(key >> 32)), key_id(key) + (uint32_t)p.v_offset[sidx]);
        cand[i] = key;
    }
    if (tid < p.n_shards) {
        const graft_vocab_partial* r = p.parts + (size_t)tid * p.rows + row;
        sC[tid] = r->c;
        sS[tid] = r->s;
        sV[tid] = r->vmax_ord;
        sN[tid] = r->nkeys;  // bit 31: a bounded wait ran out while the shard was scanned
    }
    if (tid < kMaxK) outk[tid] = 0ull;
    __syncthreads();
    // exact top-K by rank counting (keys are distinct: ids are)
    for (int i = tid; i < n; i += 128) {
        const uint64_t key = cand[i];
        if (key == 0ull) continue;
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += cand[j] > key ? 1 : 0;
        if (rank < p.K) outk[rank] = key;
    }
    __syncthreads();
    if (tid >= 32) return;
    int have = 0;
    bool internal = false;
    for (int sidx = 0; sidx < p.n_shards; ++sidx) {
        have += (int)(sN[sidx] & 0x7FFFFFFFu);
        internal = internal || (sN[sidx] >> 31) != 0u;
    }
    const int nk = have < p.K ? have : p.K;
    double Cm = -INFINITY;
    uint32_t vm = 0u;
    for (int sidx = 0; sidx < p.n_shards; ++sidx) {
        Cm = fmax(Cm, sC[sidx]);
        vm = vm > sV[sidx] ? vm : sV[sidx];
    }
    double S = 0.0;
    for (int sidx = 0; sidx < p.n_shards; ++sidx) {
        if (sC[sidx] != -INFINITY)
            S += sS[sidx] * exp2(sC[sidx] - Cm);
        else if (sS[sidx] != sS[sidx])
            S += sS[sidx];
    }
    vp_finalize(Cm, S, vm, nk, p.K, outk, lane, p.topk_id + (size_t)row * p.K, p.topk_lp + (size_t)row * p.K,
                p.lse + row, p.row_status + row, internal);
}

}  // namespace

// ---- host side ----------------------------------------------------------------------------------
static size_t vp_smem_bytes(int stages, int n_cmax) {
    return (size_t)stages * TILE + 24 * sizeof(uint64_t) + sizeof(VpShared) + (size_t)kVpBufs * n_cmax * 2 + 16;
}

VpPlan vp_make_plan(const graft_config& cfg, int num_sms, int batch) {
    VpPlan pl;
    const bool bf16 = cfg.logits_dtype == GRAFT_BF16;
    const int esz = bf16 ? 2 : 4;
    const long long nq = cfg.V / kVpQuantum > 0 ? cfg.V / kVpQuantum : 1;
    const long long Q = nq * (long long)batch * cfg.L;
    long long G = (long long)num_sms;  // one CTA per SM
    // small inputs: a CTA's share is at least 64 KiB, so that a row is not cut into more pieces than its merge is
    // worth (at batch 1 a 128 KB row over nine CTAs spent 14 us merging nine records per row)
    const long long min_share_q = (64 * 1024) / ((long long)kVpQuantum * esz);
    if (G > Q / min_share_q) G = Q / min_share_q;
    if (G > Q) G = Q;
    if (G < 1) G = 1;
    pl.grid = (int)G;
    long long share_q = (Q + G - 1) / G;
    long long seg_elems = share_q * kVpQuantum;
    seg_elems += kVpQuantum;  // a row's last quantum also takes the remainder
    if (seg_elems > cfg.V) seg_elems = cfg.V;
    pl.max_seg_tiles = (int)((seg_elems * esz + TILE - 1) / TILE) + 1;
    const size_t budget = 224 * 1024;  // one CTA per SM
    int stages = 6;
    while (stages > 2 && vp_smem_bytes(stages, pl.max_seg_tiles * NT) > budget) --stages;
    pl.stages = stages;
    pl.smem_bytes = vp_smem_bytes(stages, pl.max_seg_tiles * NT);
    return pl;
}

cudaError_t vp_launch(graft_ctx* ctx, int batch, const void* d_logits, int32_t* d_topk_id, float* d_topk_lp,
                      float* d_lse, int32_t* d_row_status, const void* d_hidden, double* d_cos,
                      graft_vocab_partial* d_partial, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    const bool bf16 = cfg.logits_dtype == GRAFT_BF16;
    VpPlan pl = vp_make_plan(cfg, ctx->num_sms, batch);
    VpParams p;
    p.logits = (const char*)d_logits;
    p.rows = batch * cfg.L;
    p.V = cfg.V;
    p.K = cfg.K;
    p.nq = cfg.V / kVpQuantum > 0 ? cfg.V / kVpQuantum : 1;
    p.Q = p.nq * p.rows;
    p.stages = pl.stages;
    p.n_cmax = pl.max_seg_tiles * NT;
    p.max_tiles = pl.max_seg_tiles;
    p.records = ctx->vp_records;
    p.row_counter = ctx->vp_row_counter;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.lse = d_lse;
    p.row_status = d_row_status;
    p.errflag = ctx->w_errflag;
    p.partial_out = d_partial;
    p.hidden = d_hidden;
    p.hidden_bf16 = cfg.hidden_dtype == GRAFT_BF16 ? 1 : 0;
    p.hidden_dim = cfg.hidden_dim;
    p.L = cfg.L;
    p.cos_out = (d_hidden != nullptr && cfg.L > 1) ? d_cos : nullptr;
    p.use_hint = 1;
    const cudaError_t e = launch_pdl(bf16 ? vocab_pass_kernel<true> : vocab_pass_kernel<false>, dim3(pl.grid),
                                     dim3(kVpThreads), pl.smem_bytes, st, p);
    ctx->launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

cudaError_t vp_merge_launch(graft_ctx* ctx, int batch, int n_shards, const graft_vocab_partial* d_parts,
                            const int32_t* h_v_offset, int32_t* d_topk_id, float* d_topk_lp, float* d_lse,
                            int32_t* d_row_status, cudaStream_t st) {
    MergeParams p;
    p.parts = d_parts;
    p.n_shards = n_shards;
    p.rows = batch * ctx->cfg.L;
    p.K = ctx->cfg.K;
    for (int i = 0; i < kMergeMaxShards; ++i) p.v_offset[i] = i < n_shards ? h_v_offset[i] : 0;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.lse = d_lse;
    p.row_status = d_row_status;
    vocab_merge_kernel<<<p.rows, 128, 0, st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}
int vp_merge_max_shards() { return kMergeMaxShards; }

cudaError_t vp_configure(const graft_config& cfg, int num_sms, size_t* max_smem) {
    // the largest dynamic shared-memory request any batch can produce (segment = a whole row)
    VpPlan pl = vp_make_plan(cfg, num_sms, cfg.max_batch > 4096 ? cfg.max_batch : 4096);
    *max_smem = pl.smem_bytes;
    if (pl.smem_bytes > 225 * 1024) return cudaErrorInvalidValue;
    cudaError_t e;
    if (cfg.logits_dtype == GRAFT_BF16)
        e = cudaFuncSetAttribute(vocab_pass_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
    else
        e = cudaFuncSetAttribute(vocab_pass_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024);
    return e;
}

}  // namespace graft

// ---- allocation-free variant of the vocab pass ------------------------------------------------------------
// Some callers cannot let this library allocate: a serving process that handed all device memory to its own
// pool at start-up (a cudaMalloc there fails, or stalls every stream while the driver synchronises), or code
// that must stay off the driver's allocation lock on its latency path.  For them the scratch of the vocab
// pass -- the per-CTA records of rows shared between CTAs, the per-row arrival counters and the error word --
// lives in the file-scope device array below instead of a context's cudaMalloc'ed workspace.  Every GPU that
// loads this library holds the array (about 0.4 MB) until the process exits.
namespace graft {
namespace {

constexpr int kStaticMaxGrid = 512;     // CTAs (one per SM is launched): room for any device
constexpr int kStaticMaxRows = 16384;   // batch * L

struct VpStaticScratch {
    VpRecord records[kStaticMaxGrid * 2];
    int row_counter[kStaticMaxRows];
    int errflag[64];
};

static __device__ __align__(256) unsigned char g_vp_static_scratch[sizeof(VpStaticScratch)];

struct VpStaticDevice {
    bool ready = false;
    VpStaticScratch* scratch = nullptr;  // device address of g_vp_static_scratch on this device
    int num_sms = 0;
};
VpStaticDevice g_vp_static_dev[64];
std::mutex g_vp_static_mutex;

}  // namespace
}  // namespace graft

extern "C" graft_status graft_vocab_pass_static(int32_t batch, int32_t L, int32_t V, int32_t K,
                                                graft_dtype logits_dtype, const void* d_logits, int32_t* d_topk_id,
                                                float* d_topk_lp, float* d_lse, int32_t* d_row_status, void* stream) {
    using namespace graft;
    if (!d_logits || !d_topk_id || !d_topk_lp || !d_lse || !d_row_status) return GRAFT_ERR_INVALID_ARG;
    if (logits_dtype != GRAFT_F32 && logits_dtype != GRAFT_BF16) return GRAFT_ERR_INVALID_ARG;
    if (batch < 1 || L < 1 || V < 1 || K < 1) return GRAFT_ERR_INVALID_ARG;
    if ((uintptr_t)d_logits % (logits_dtype == GRAFT_BF16 ? 2 : 4)) return GRAFT_ERR_INVALID_ARG;
    if (K > kMaxK || K > V || L > kMaxL || (long long)V > 2147483647LL - 64) return GRAFT_ERR_UNSUPPORTED;
    if ((long long)batch * L > kStaticMaxRows) return GRAFT_ERR_UNSUPPORTED;  // beyond the static scratch
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    graft_config cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.V = V;
    cfg.L = L;
    cfg.K = K;
    cfg.max_batch = batch;
    cfg.logits_dtype = logits_dtype;
    VpStaticDevice* sd = &g_vp_static_dev[dev];
    {
        // set-up, once per device, with that device current: the array's name is only a host-side stand-in
        // here, so its device address has to be asked for
        std::lock_guard<std::mutex> lock(g_vp_static_mutex);
        if (!sd->ready) {
            void* ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_vp_static_scratch) != cudaSuccess || !ptr) {
                cudaGetLastError();
                return GRAFT_ERR_CUDA;
            }
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
                cudaGetLastError();
                return GRAFT_ERR_CUDA;
            }
            if (cudaFuncSetAttribute(vocab_pass_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) !=
                    cudaSuccess ||
                cudaFuncSetAttribute(vocab_pass_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) !=
                    cudaSuccess) {
                cudaGetLastError();
                return GRAFT_ERR_CUDA;
            }
            sd->scratch = (VpStaticScratch*)ptr;
            sd->num_sms = sms;
            sd->ready = true;
        }
    }
    const VpPlan pl = vp_make_plan(cfg, sd->num_sms, batch);
    if (pl.grid > kStaticMaxGrid || pl.smem_bytes > 225 * 1024) return GRAFT_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the arrival counters and the error word must start at 0
    if (cudaMemsetAsync(sd->scratch->row_counter, 0, sizeof(int) * (size_t)batch * L, st) != cudaSuccess ||
        cudaMemsetAsync(sd->scratch->errflag, 0, sizeof(sd->scratch->errflag), st) != cudaSuccess) {
        cudaGetLastError();
        return GRAFT_ERR_CUDA;
    }
    VpParams p;
    p.logits = (const char*)d_logits;
    p.rows = batch * L;
    p.V = V;
    p.K = K;
    p.nq = V / kVpQuantum > 0 ? V / kVpQuantum : 1;
    p.Q = p.nq * p.rows;
    p.stages = pl.stages;
    p.n_cmax = pl.max_seg_tiles * NT;
    p.max_tiles = pl.max_seg_tiles;
    p.records = sd->scratch->records;
    p.row_counter = sd->scratch->row_counter;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.lse = d_lse;
    p.row_status = d_row_status;
    p.errflag = sd->scratch->errflag;
    p.partial_out = nullptr;
    p.hidden = nullptr;
    p.hidden_bf16 = 0;
    p.hidden_dim = 0;
    p.L = L;
    p.cos_out = nullptr;
    p.use_hint = 1;
    if (logits_dtype == GRAFT_BF16)
        vocab_pass_kernel<true><<<pl.grid, kVpThreads, pl.smem_bytes, st>>>(p);
    else
        vocab_pass_kernel<false><<<pl.grid, kVpThreads, pl.smem_bytes, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? GRAFT_OK : GRAFT_ERR_CUDA;
}
