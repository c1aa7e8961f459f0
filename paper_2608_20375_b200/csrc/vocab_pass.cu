// Vocab pass: for every (sequence, future position) row of the drafter logits, one streaming read that
// yields log-sum-exp over the vocabulary and the K top-ranked tokens with their log-probabilities
// (Preliminaries, "DFlash one-pass marginals": q_{t,d} and c^{(r)}_{t,d}; Eq. 3's log q).
//
// Shape of the kernel (sm_100a):
//   * persistent grid, two CTAs per SM; the rows*V element stream is cut into equal contiguous shares,
//     one per CTA, so a CTA sees at most two partial rows plus whole rows in between;
//   * one producer warp feeds a shared-memory ring with 16 KiB TMA bulk copies (cp.async.bulk +
//     mbarrier complete_tx); eight consumer warps read the ring with 16-byte shared loads;
//   * per 32-element chunk a consumer lane takes a packed max (stored for the second stage, 2 bytes per
//     chunk), keeps a lazily rescaled reference exponent and adds 2^(z log2e - ref) with ex2.approx;
//   * top-K needs no per-element work in the stream: after the segment, the K-th largest per-thread
//     maximum is a lower bound T for the K-th largest element; only chunks whose stored max reaches T
//     (about K of them) are re-read, their elements >= T become 64-bit keys (value desc, id asc) and the
//     exact top-K is found by rank counting.  An overflow of the small key buffer (adversarial rows)
//     falls back to an exact chunked selection;
//   * rows shared by several CTAs are merged by the last CTA to arrive (a counter, no waiting).
#include "common.cuh"
#include "internal.h"

namespace graft {

namespace {

constexpr int NW = kVpConsumerWarps;
constexpr int NT = kVpConsumers;
constexpr int TILE = kVpTileBytes;
constexpr int WBLK = TILE / NW;  // bytes of a tile owned by one warp (2048)
constexpr int VEC_PER_LANE = WBLK / 16 / 32;  // 4
constexpr int CONS_BAR = 1;
static_assert(VEC_PER_LANE == 4, "chunk layout assumes four 16-byte vectors per lane per tile");

template <bool BF16>
struct VT;
template <>
struct VT<true> {
    using cm_t = uint16_t;
    static constexpr int ESZ = 2, EPV = 8, CH = 32;
    static constexpr uint32_t NEG_INF_WORD = 0xFF80FF80u;
};
template <>
struct VT<false> {
    using cm_t = uint32_t;
    static constexpr int ESZ = 4, EPV = 4, CH = 16;
    static constexpr uint32_t NEG_INF_WORD = 0xFF800000u;
};

struct VpParams {
    const char* logits;
    int rows, V, K;
    long long nq;  // quanta per row
    long long Q;   // quanta in total
    int stages;
    int n_cmax;    // chunk-max slots in shared memory
    VpRecord* records;
    int* row_counter;
    int32_t* topk_id;
    float* topk_lp;
    float* lse;
    int32_t* row_status;
    int32_t* errflag;
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

template <bool BF16>
__device__ __forceinline__ Seg make_seg(const VpParams& p, long long qi, long long qend) {
    using T = VT<BF16>;
    Seg s;
    s.row = (int)(qi / p.nq);
    long long qr0 = qi - (long long)s.row * p.nq;
    long long qr1 = qr0 + (qend - qi);
    if (qr1 > p.nq) qr1 = p.nq;
    s.e0 = (int)(qr0 * kVpQuantum);
    long long e1 = qr1 * kVpQuantum;
    s.e1 = e1 > p.V ? p.V : (int)e1;
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

__device__ __forceinline__ float load_elem_f32(const char* p, bool bf16) {
    if (bf16) return __uint_as_float(((uint32_t) * (const uint16_t*)p) << 16);
    return *(const float*)p;
}

// ---- per-thread streaming state -----------------------------------------------------------------
struct Acc {
    float ref;     // reference exponent, log2 domain; -inf before the first finite value
    float s;       // sum of 2^(z log2e - ref)
    uint32_t tmo;  // ord() of the largest value seen; 0 = nothing seen
};

__device__ __forceinline__ float acc_begin_chunk(Acc& a, float cm) {
    // Raise the reference only when the chunk maximum exceeds it by more than 2^16: rescaling is then
    // rare, and every term stays below 2^16.
    float cms = cm * kLog2e;
    if (cms > a.ref + 16.0f) {
        a.s *= ex2_approx(a.ref - cms);
        a.ref = cms;
    }
    return (a.ref == -INFINITY) ? 0.0f : -a.ref;
}

template <bool BF16, bool GUARD>
__device__ __forceinline__ void process_chunk(const uint4* __restrict__ wb, int lane, int nvalid_vec, Acc& a,
                                              typename VT<BF16>::cm_t* cmax_slot) {
    using T = VT<BF16>;
    uint4 v[VEC_PER_LANE];
#pragma unroll
    for (int i = 0; i < VEC_PER_LANE; ++i) {
        if (!GUARD || (i * 32 + lane) < nvalid_vec)
            v[i] = wb[i * 32 + lane];
        else
            v[i] = make_uint4(T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD, T::NEG_INF_WORD);
    }
    float cm;
    if (BF16) {
        uint32_t m0 = hmax2_bf16(hmax2_bf16(v[0].x, v[0].y), hmax2_bf16(v[0].z, v[0].w));
        uint32_t m1 = hmax2_bf16(hmax2_bf16(v[1].x, v[1].y), hmax2_bf16(v[1].z, v[1].w));
        uint32_t m2 = hmax2_bf16(hmax2_bf16(v[2].x, v[2].y), hmax2_bf16(v[2].z, v[2].w));
        uint32_t m3 = hmax2_bf16(hmax2_bf16(v[3].x, v[3].y), hmax2_bf16(v[3].z, v[3].w));
        uint32_t pm = hmax2_bf16(hmax2_bf16(m0, m1), hmax2_bf16(m2, m3));
        cm = fmaxf(__uint_as_float(pm << 16), __uint_as_float(pm & 0xFFFF0000u));
        *cmax_slot = (typename T::cm_t)(__float_as_uint(cm) >> 16);
    } else {
        float m = -INFINITY;
#pragma unroll
        for (int i = 0; i < VEC_PER_LANE; ++i) {
            m = fmaxf(m, fmaxf(fmaxf(__uint_as_float(v[i].x), __uint_as_float(v[i].y)),
                               fmaxf(__uint_as_float(v[i].z), __uint_as_float(v[i].w))));
        }
        cm = m;
        *cmax_slot = (typename T::cm_t)__float_as_uint(cm);
    }
    uint32_t o = ord_from_float(cm);
    a.tmo = o > a.tmo ? o : a.tmo;
    const float nref = acc_begin_chunk(a, cm);
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int i = 0; i < VEC_PER_LANE; ++i) {
        const uint32_t w[4] = {v[i].x, v[i].y, v[i].z, v[i].w};
        if (BF16) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xFFFF0000u);
                float e0 = ex2_approx(fmaf(lo, kLog2e, nref)), e1 = ex2_approx(fmaf(hi, kLog2e, nref));
                if (k & 1) {
                    s2 += e0;
                    s3 += e1;
                } else {
                    s0 += e0;
                    s1 += e1;
                }
            }
        } else {
            s0 += ex2_approx(fmaf(__uint_as_float(w[0]), kLog2e, nref));
            s1 += ex2_approx(fmaf(__uint_as_float(w[1]), kLog2e, nref));
            s2 += ex2_approx(fmaf(__uint_as_float(w[2]), kLog2e, nref));
            s3 += ex2_approx(fmaf(__uint_as_float(w[3]), kLog2e, nref));
        }
    }
    a.s += (s0 + s1) + (s2 + s3);
}

// ---- shared-memory control block ---------------------------------------------------------------
struct __align__(16) VpShared {
    uint64_t cand[kVpCandCap];
    uint64_t outk[kMaxK];
    uint32_t hits[kVpHitCap];
    uint32_t tmax[NT];
    float wc[NW], ws[NW];
    uint32_t wv[NW];
    int ncand, nhits, overflow;
    uint32_t T;
    float segC, segS;
    uint32_t segV;
    int is_last;
    volatile int abort_flag;
};

__device__ __forceinline__ void cons_bar() { named_bar_sync(CONS_BAR, NT); }

// Exact top-K of cand[0..n) by rank counting; result sorted descending in outk[0..min(n,K)).
// Keys are distinct (ids are), so ranks are a permutation.  Ends with a consumer barrier.
__device__ void select_topk(VpShared* sh, int n, int K, int tid) {
    for (int i = tid; i < n; i += NT) {
        const uint64_t key = sh->cand[i];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (sh->cand[j] > key) ? 1 : 0;
        if (rank < K) sh->outk[rank] = key;
    }
    cons_bar();
}

// Exact selection over a whole segment straight from global memory, in slices small enough that the key
// buffer cannot overflow.  Used only when the fast path's buffers overflowed.
template <bool BF16>
__device__ void fallback_select(VpShared* sh, const VpParams& p, const Seg& sg, int tid, int* nk_out) {
    using T = VT<BF16>;
    const int K = p.K;
    const int slice = kVpCandCap - kMaxK;
    const char* rowp = p.logits + (size_t)sg.row * p.V * T::ESZ;
    uint64_t thr = 0;
    int nb = 0;
    for (int base = sg.e0; base < sg.e1; base += slice) {
        if (tid == 0) sh->ncand = nb;
        cons_bar();
        int end = base + slice < sg.e1 ? base + slice : sg.e1;
        for (int e = base + tid; e < end; e += NT) {
            float x = load_elem_f32(rowp + (size_t)e * T::ESZ, BF16);
            uint64_t key = make_key(__float_as_uint(x), (uint32_t)e);
            if (key > thr) {
                int pos = atomicAdd(&sh->ncand, 1);
                sh->cand[pos] = key;
            }
        }
        cons_bar();
        int n = sh->ncand;
        if (n > K) {
            select_topk(sh, n, K, tid);
            if (tid < K) sh->cand[tid] = sh->outk[tid];
            thr = sh->outk[K - 1];
            nb = K;
            cons_bar();
        } else {
            nb = n;
        }
    }
    select_topk(sh, nb, K, tid);
    *nk_out = nb < K ? nb : K;
}

template <bool BF16>
__global__ void __launch_bounds__(kVpThreads, 2) vocab_pass_kernel(const VpParams p) {
    using T = VT<BF16>;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    unsigned char* ring = smem_raw;
    uint64_t* bars = (uint64_t*)(ring + (size_t)p.stages * TILE);
    VpShared* sh = (VpShared*)(bars + 2 * 8);
    typename T::cm_t* cmax = (typename T::cm_t*)(sh + 1);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const long long G = gridDim.x;
    const long long q0 = cta_start(blockIdx.x, p.Q, G), q1 = cta_start(blockIdx.x + 1, p.Q, G);
    const uint32_t full0 = smem_u32(bars), empty0 = smem_u32(bars + 8);

    if (tid == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full0 + 8 * s, 1);
            mbar_init(empty0 + 8 * s, NW);
        }
        mbar_fence_init();
        sh->ncand = 0;
        sh->nhits = 0;
        sh->overflow = 0;
        sh->abort_flag = 0;
    }
    __syncthreads();

    if (warp == NW) {
        // ------------------------------ producer warp --------------------------------------------
        if (lane == 0) {
            uint64_t policy = 0;
            if (p.use_hint) policy = l2_policy_evict_first();
            uint32_t t = 0, st = 0, ph = 1;  // ph: parity of the "empty" phase to wait for (first lap: none)
            const uint32_t nst = (uint32_t)p.stages;
            for (long long qi = q0; qi < q1;) {
                Seg sg = make_seg<BF16>(p, qi, q1);
                qi += (sg.e1 - sg.e0 + kVpQuantum - 1) / kVpQuantum;
                for (int tile = 0; tile < sg.ntiles; ++tile, ++t) {
                    if (t >= nst) mbar_wait_bounded(empty0 + 8 * st, ph, &sh->abort_flag);
                    uint32_t off = (uint32_t)tile * TILE;
                    uint32_t bytes = sg.body_bytes - off < (uint32_t)TILE ? sg.body_bytes - off : (uint32_t)TILE;
                    mbar_arrive_expect_tx(full0 + 8 * st, bytes);
                    if (p.use_hint)
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
                for (uint32_t back = 0; back < (uint32_t)p.stages && back < t; ++back) {
                    uint32_t tt = t - 1 - back;
                    uint32_t tries = 0;
                    while (!mbar_try_wait(full0 + 8 * (tt % p.stages), (tt / p.stages) & 1) && ++tries < GRAFT_SPIN_LIMIT) {
                    }
                }
            }
        }
    } else {
        // ------------------------------ consumer warps -------------------------------------------
        uint32_t st = 0, ph = 0;  // ring position and parity of the "full" phase to wait for
        const uint32_t nst = (uint32_t)p.stages;
        for (long long qi = q0; qi < q1;) {
            const Seg sg = make_seg<BF16>(p, qi, q1);
            qi += (sg.e1 - sg.e0 + kVpQuantum - 1) / kVpQuantum;
            const char* rowp = p.logits + (size_t)sg.row * p.V * T::ESZ;
            Acc a;
            a.ref = -INFINITY;
            a.s = 0.f;
            a.tmo = 0u;

            // ragged head / tail that the 16-byte bulk copies cannot carry: plain loads, every element a candidate
            {
                const int nhead = sg.e_body0 - sg.e0, ntail = sg.e1 - sg.e_tail0;
                for (int i = tid; i < nhead + ntail; i += NT) {
                    const int e = i < nhead ? sg.e0 + i : sg.e_tail0 + (i - nhead);
                    const float x = load_elem_f32(rowp + (size_t)e * T::ESZ, BF16);
                    uint32_t o = ord_from_float(x);
                    a.tmo = o > a.tmo ? o : a.tmo;
                    const float nref = acc_begin_chunk(a, x);
                    a.s += ex2_approx(fmaf(x, kLog2e, nref));
                    int pos = atomicAdd(&sh->ncand, 1);
                    if (pos < kVpCandCap)
                        sh->cand[pos] = make_key(__float_as_uint(x), (uint32_t)e);
                    else
                        sh->overflow = 1;
                }
            }

            {
                const int nfull = (int)(sg.body_bytes / TILE);
                typename T::cm_t* slot = cmax + tid;
                for (int tile = 0; tile < sg.ntiles; ++tile, slot += NT) {
                    mbar_wait_bounded(full0 + 8 * st, ph, &sh->abort_flag);
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

            // ---------------- segment epilogue -------------------------------------------------------
            // E1: per-thread maxima to shared memory; (ref, s) and the maximum reduced per warp
            sh->tmax[tid] = a.tmo;
            {
                float c = a.ref, s = a.s;
                uint32_t vm = a.tmo;
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) {
                    float c2 = __shfl_xor_sync(0xFFFFFFFFu, c, d);
                    float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, d);
                    uint32_t v2 = __shfl_xor_sync(0xFFFFFFFFu, vm, d);
                    float cn = fmaxf(c, c2);
                    float f1 = (c == -INFINITY) ? 0.f : ex2_approx(c - cn);
                    float f2 = (c2 == -INFINITY) ? 0.f : ex2_approx(c2 - cn);
                    s = s * f1 + s2 * f2;
                    c = cn;
                    vm = vm > v2 ? vm : v2;
                }
                if (lane == 0) {
                    sh->wc[warp] = c;
                    sh->ws[warp] = s;
                    sh->wv[warp] = vm;
                }
            }
            cons_bar();
            // E2: warp 0 finds T = the K-th largest per-thread maximum, truncated to its top 16 bits
            //     (a lower bound of the K-th largest element); warp 1 folds the warps' (ref, s).
            if (warp == 0) {
                uint32_t mine[NT / 32];
#pragma unroll
                for (int i = 0; i < NT / 32; ++i) mine[i] = sh->tmax[i * 32 + lane];
                uint32_t Tv = 0;
                for (int bit = 31; bit >= 16; --bit) {
                    const uint32_t trial = Tv | (1u << bit);
                    int cnt = 0;
#pragma unroll
                    for (int i = 0; i < NT / 32; ++i) cnt += (mine[i] >= trial) ? 1 : 0;
                    cnt = __reduce_add_sync(0xFFFFFFFFu, cnt);
                    if (cnt >= p.K) Tv = trial;
                }
                if (lane == 0) sh->T = Tv;
            } else if (warp == 1) {
                float c = lane < NW ? sh->wc[lane] : -INFINITY;
                float s = lane < NW ? sh->ws[lane] : 0.f;
                uint32_t vm = lane < NW ? sh->wv[lane] : 0u;
#pragma unroll
                for (int d = NW / 2; d > 0; d >>= 1) {
                    float c2 = __shfl_xor_sync(0xFFFFFFFFu, c, d);
                    float s2 = __shfl_xor_sync(0xFFFFFFFFu, s, d);
                    uint32_t v2 = __shfl_xor_sync(0xFFFFFFFFu, vm, d);
                    float cn = fmaxf(c, c2);
                    float f1 = (c == -INFINITY) ? 0.f : ex2_approx(c - cn);
                    float f2 = (c2 == -INFINITY) ? 0.f : ex2_approx(c2 - cn);
                    s = s * f1 + s2 * f2;
                    c = cn;
                    vm = vm > v2 ? vm : v2;
                }
                if (lane == 0) {
                    sh->segC = c;
                    sh->segS = s;
                    sh->segV = vm;
                }
            }
            cons_bar();
            // E3: every thread scans the chunk maxima it stored itself
            {
                const uint32_t Tv = sh->T;
                for (int tile = 0; tile < sg.ntiles; ++tile) {
                    const uint32_t cs = (uint32_t)tile * NT + tid;
                    const uint32_t bits = BF16 ? ((uint32_t)cmax[cs] << 16) : (uint32_t)cmax[cs];
                    if (ord_from_bits(bits) >= Tv) {
                        int pos = atomicAdd(&sh->nhits, 1);
                        if (pos < kVpHitCap)
                            sh->hits[pos] = cs;
                        else
                            sh->overflow = 1;
                    }
                }
            }
            cons_bar();
            // E4: elements of the hit chunks, one element per thread and step, re-read from global memory
            {
                const uint32_t Tv = sh->T;
                const int nh = sh->nhits < kVpHitCap ? sh->nhits : kVpHitCap;
                for (int idx = tid; idx < nh * T::CH; idx += NT) {
                    const uint32_t cs = sh->hits[idx / T::CH];
                    const int j = idx % T::CH;
                    const uint32_t tile = cs / NT, r = cs % NT, w = r >> 5, l = r & 31;
                    const uint32_t off = tile * TILE + w * WBLK + ((j / T::EPV) * 32 + l) * 16 + (j % T::EPV) * T::ESZ;
                    if (off < sg.body_bytes) {
                        const float x = load_elem_f32(sg.body + off, BF16);
                        if (ord_from_float(x) >= Tv) {
                            int pos = atomicAdd(&sh->ncand, 1);
                            if (pos < kVpCandCap)
                                sh->cand[pos] = make_key(__float_as_uint(x), (uint32_t)(sg.e_body0 + off / T::ESZ));
                            else
                                sh->overflow = 1;
                        }
                    }
                }
            }
            cons_bar();
            // E5: exact top-K of the candidates
            int nk;
            if (sh->overflow) {
                fallback_select<BF16>(sh, p, sg, tid, &nk);
            } else {
                const int n = sh->ncand;
                select_topk(sh, n, p.K, tid);
                nk = n < p.K ? n : p.K;
            }
            // E6: finish the row, or leave a record for the CTA that arrives last
            const long long x0 = (long long)sg.row * p.nq;
            const int c_first = cta_of(x0, p.Q, G), c_last = cta_of(x0 + p.nq - 1, p.Q, G);
            const int nseg = c_last - c_first + 1;
            double Cd = (double)sh->segC, Sd = (double)sh->segS;
            uint32_t Vm = sh->segV;
            bool finish = (nseg == 1);
            if (nseg > 1) {
                const int my_first_row = (int)(q0 / p.nq);
                VpRecord* rec = p.records + (size_t)blockIdx.x * 2 + (sg.row == my_first_row ? 0 : 1);
                if (tid < kMaxK) rec->keys[tid] = tid < nk ? sh->outk[tid] : 0ull;
                if (tid == 0) {
                    rec->c = sh->segC;
                    rec->s = sh->segS;
                    rec->vmax = __uint_as_float(sh->segV);
                    rec->nkeys = (uint32_t)nk;
                }
                __threadfence();
                cons_bar();
                if (tid == 0) {
                    int old = atomicAdd(p.row_counter + sg.row, 1);
                    sh->is_last = (old == nseg - 1);
                    __threadfence();
                }
                cons_bar();
                if (sh->is_last) {
                    finish = true;
                    // merge the records of CTAs c_first..c_last, a round at a time
                    const int per_round = (kVpCandCap - kMaxK) / kMaxK;
                    int have = 0;
                    for (int c0 = c_first; c0 <= c_last; c0 += per_round) {
                        const int c1 = c0 + per_round - 1 < c_last ? c0 + per_round - 1 : c_last;
                        if (tid == 0) sh->ncand = have;
                        cons_bar();
                        for (int i = tid; i < (c1 - c0 + 1) * kMaxK; i += NT) {
                            const int c = c0 + i / kMaxK, k = i % kMaxK;
                            const int c_row0 = (int)(cta_start(c, p.Q, G) / p.nq);
                            const VpRecord* r = p.records + (size_t)c * 2 + (sg.row == c_row0 ? 0 : 1);
                            const uint64_t key = __ldcg((const unsigned long long*)&r->keys[k]);
                            if (key != 0ull) sh->cand[atomicAdd(&sh->ncand, 1)] = key;
                        }
                        cons_bar();
                        const int n = sh->ncand;
                        select_topk(sh, n, p.K, tid);
                        have = n < p.K ? n : p.K;
                        if (tid < have) sh->cand[tid] = sh->outk[tid];
                        cons_bar();
                    }
                    nk = have;
                    // log-sum-exp pieces, folded in double by one thread per record and a warp reduction
                    if (warp == 0) {
                        double Cm = -INFINITY;
                        uint32_t vm = 0;
                        for (int c = c_first + lane; c <= c_last; c += 32) {
                            const int c_row0 = (int)(cta_start(c, p.Q, G) / p.nq);
                            const VpRecord* r = p.records + (size_t)c * 2 + (sg.row == c_row0 ? 0 : 1);
                            float rc = __ldcg(&r->c);
                            uint32_t rv = __float_as_uint(__ldcg(&r->vmax));
                            Cm = fmax(Cm, (double)rc);
                            vm = vm > rv ? vm : rv;
                        }
#pragma unroll
                        for (int d = 16; d > 0; d >>= 1) {
                            Cm = fmax(Cm, __shfl_xor_sync(0xFFFFFFFFu, Cm, d));
                            uint32_t v2 = __shfl_xor_sync(0xFFFFFFFFu, vm, d);
                            vm = vm > v2 ? vm : v2;
                        }
                        double S = 0.0;
                        for (int c = c_first + lane; c <= c_last; c += 32) {
                            const int c_row0 = (int)(cta_start(c, p.Q, G) / p.nq);
                            const VpRecord* r = p.records + (size_t)c * 2 + (sg.row == c_row0 ? 0 : 1);
                            float rc = __ldcg(&r->c), rs = __ldcg(&r->s);
                            if (rc != -INFINITY) S += (double)rs * exp2((double)rc - Cm);
                            else if (rs != rs) S += (double)rs;
                        }
#pragma unroll
                        for (int d = 16; d > 0; d >>= 1) S += __shfl_xor_sync(0xFFFFFFFFu, S, d);
                        if (lane == 0) {
                            sh->segC = (float)Cm;  // exact: Cm is one of the fp32 references
                            sh->segS = (float)S;
                            sh->segV = vm;
                        }
                        Cd = Cm;
                        Sd = S;
                        Vm = vm;
                    }
                    if (tid == 0) p.row_counter[sg.row] = 0;
                }
            }
            if (finish && warp == 0) {
                // lse = (C + log2 S) ln 2, in double; every lane of warp 0 holds the same Cd, Sd, Vm
                // The stream accumulates 2^(z c - ref) with c = fp32(log2 e), so (C + log2 S) ln 2 is the
                // log-sum-exp of the logits scaled by a = c ln 2 = 1 + 1.3e-8.  To first order that adds
                // (a - 1) E_q[z]; the largest logit stands in for the mean under q (the difference is a few
                // units times 1e-8).
                const float vmax = __uint_as_float(bits_from_ord(Vm));
                const double a_minus_1 = (double)kLog2e * kLn2 - 1.0;
                const double lse_d = (Cd + log2(Sd)) * kLn2 - a_minus_1 * (double)vmax;
                const float lse_f = (float)lse_d;
                const bool bad = !(Sd > 0.0) || !(Sd < 1e300) || Vm == 0u || vmax == INFINITY || vmax == -INFINITY ||
                                 nk < p.K;
                if (lane < p.K) {
                    const uint64_t key = lane < nk ? sh->outk[lane] : 0ull;
                    p.topk_id[(size_t)sg.row * p.K + lane] = lane < nk ? (int32_t)key_id(key) : -1;
                    p.topk_lp[(size_t)sg.row * p.K + lane] = lane < nk ? (float)((double)key_value(key) - lse_d) : 0.f;
                }
                if (lane == 0) {
                    p.lse[sg.row] = lse_f;
                    p.row_status[sg.row] = bad ? GRAFT_ST_BAD_LOGITS : 0;
                }
            }
            // E7: reset the counters for the next segment
            if (tid == 0) {
                sh->ncand = 0;
                sh->nhits = 0;
                sh->overflow = 0;
            }
            cons_bar();
        }
    }
    __syncthreads();
    if (tid == 0 && sh->abort_flag) atomicOr(p.errflag, 1);
}

}  // namespace

// ---- host side ----------------------------------------------------------------------------------
static size_t vp_smem_bytes(int stages, int n_cmax, bool bf16) {
    return (size_t)stages * TILE + 16 * sizeof(uint64_t) + sizeof(VpShared) + (size_t)n_cmax * (bf16 ? 2 : 4) + 16;
}

VpPlan vp_make_plan(const graft_config& cfg, int num_sms, int batch) {
    VpPlan pl;
    const bool bf16 = cfg.logits_dtype == GRAFT_BF16;
    const int esz = bf16 ? 2 : 4;
    const long long nq = ((long long)cfg.V + kVpQuantum - 1) / kVpQuantum;
    const long long Q = nq * (long long)batch * cfg.L;
    long long G = (long long)num_sms * 2;
    if (G > Q) G = Q;
    if (G < 1) G = 1;
    pl.grid = (int)G;
    long long share_q = (Q + G - 1) / G;
    long long seg_elems = share_q * kVpQuantum;
    if (seg_elems > nq * kVpQuantum) seg_elems = nq * kVpQuantum;
    pl.max_seg_tiles = (int)((seg_elems * esz + TILE - 1) / TILE) + 1;
    const size_t budget = 112 * 1024;  // two CTAs per SM
    int stages = 6;
    while (stages > 2 && vp_smem_bytes(stages, pl.max_seg_tiles * NT, bf16) > budget) --stages;
    pl.stages = stages;
    pl.smem_bytes = vp_smem_bytes(stages, pl.max_seg_tiles * NT, bf16);
    return pl;
}

cudaError_t vp_launch(graft_ctx* ctx, int batch, const void* d_logits, int32_t* d_topk_id, float* d_topk_lp,
                      float* d_lse, int32_t* d_row_status, cudaStream_t st) {
    const graft_config& cfg = ctx->cfg;
    const bool bf16 = cfg.logits_dtype == GRAFT_BF16;
    VpPlan pl = vp_make_plan(cfg, ctx->num_sms, batch);
    VpParams p;
    p.logits = (const char*)d_logits;
    p.rows = batch * cfg.L;
    p.V = cfg.V;
    p.K = cfg.K;
    p.nq = ((long long)cfg.V + kVpQuantum - 1) / kVpQuantum;
    p.Q = p.nq * p.rows;
    p.stages = pl.stages;
    p.n_cmax = pl.max_seg_tiles * NT;
    p.records = ctx->vp_records;
    p.row_counter = ctx->vp_row_counter;
    p.topk_id = d_topk_id;
    p.topk_lp = d_topk_lp;
    p.lse = d_lse;
    p.row_status = d_row_status;
    p.errflag = ctx->w_errflag;
    p.use_hint = 1;
    if (bf16)
        vocab_pass_kernel<true><<<pl.grid, kVpThreads, pl.smem_bytes, st>>>(p);
    else
        vocab_pass_kernel<false><<<pl.grid, kVpThreads, pl.smem_bytes, st>>>(p);
    ctx->launches += 1;
    return cudaGetLastError();
}

cudaError_t vp_configure(const graft_config& cfg, int num_sms, size_t* max_smem) {
    // the largest dynamic shared-memory request any batch can produce (segment = a whole row)
    VpPlan pl = vp_make_plan(cfg, num_sms, cfg.max_batch > 4096 ? cfg.max_batch : 4096);
    *max_smem = pl.smem_bytes;
    if (pl.smem_bytes > 113 * 1024 && pl.stages <= 2) return cudaErrorInvalidValue;
    cudaError_t e;
    if (cfg.logits_dtype == GRAFT_BF16)
        e = cudaFuncSetAttribute(vocab_pass_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 114 * 1024);
    else
        e = cudaFuncSetAttribute(vocab_pass_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 114 * 1024);
    return e;
}

}  // namespace graft
