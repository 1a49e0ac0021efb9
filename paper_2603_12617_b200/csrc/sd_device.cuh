// Device-side building blocks of the verify-and-feedback kernels (sm_100a).
//
// Arithmetic contract shared by every kernel in this library, so that a value recomputed later
// (the in-chunk inverse-CDF search) is bit-identical to the value summed earlier:
//   c      = fp32(log2(e)/tau)
//   e_v    = ex2.approx.ftz( fma(z_v, c, -R) ),  R = fl(m*c), m = row maximum
//   g_v    = fma(eD_v, kD, -(eT_v*kT)),          kX = fp32((1/tau)/S_X)       [ = (q-p)/tau ]
//   r_v    = max(0, -g_v)                                                      [ = max(0,p-q)/tau ]
//   bonus row: r_v = eT_v * kT with kT = fp32(1/S_T)                           [ = p ]
// Row scalars (S, the KL accumulator, log-sum-exp, the accept ratio, CDF prefixes) are combined
// in fp64 in a fixed order, so results do not depend on scheduling.
#pragma once

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sd_verify.h"

namespace sdv {

namespace cg = cooperative_groups;

constexpr int kWarps = 8;
constexpr int kThreads = kWarps * 32;
constexpr int kChunkVecs = 128;                  // 16-byte vectors of one row in a sampling chunk
constexpr int kChunkBytes = kChunkVecs * 16;     // 2 KiB of one row
constexpr int kPieceChunks = 4;                  // sampling chunks fetched by one bulk copy
constexpr int kMaxPieces = 16;                   // bulk copies (per row) a block may issue
constexpr int kMaxChunksPerBlock = kMaxPieces * kPieceChunks;
constexpr int kMaxCluster = 16;
constexpr uint32_t kStatusTimeout = 0x80000000u; // internal: a bounded wait gave up
constexpr uint32_t kWaitLimit = 1u << 22;        // polls of an mbarrier before giving up

// Constants a finished row leaves behind for the inverse-CDF search.
struct __align__(16) RowConst {
    float negRT;  // -fl(mT*c)
    float negRD;  // -fl(mD*c)
    float kT;     // pair row: (1/tau)/S_T ; bonus row: 1/S_T
    float kD;     // pair row: (1/tau)/S_D ; bonus row: 0
};

// Softmax statistics of a slice of one row pair.
struct PartialStats {
    float mT, mD;      // slice maxima (raw logits); -FLT_MAX for an empty slice
    double sT, sD;     // sum of ex2(fma(z,c,-fl(m*c)))
    double w;          // sum of eT*((t-mT)-(d-mD)), same reference as sT
};

struct Params {
    const void* T;           // [B,k+1,V]
    const void* D;           // [B,k,V]
    const int32_t* x;        // [B,k]
    const float* u;          // [B,k+1]
    int B, k, V;
    int NC;                  // sampling chunks per row
    float c;                 // fp32(log2e/tau)
    float tau;
    double c64;              // log2e/tau
    double inv_tau;
    // outputs
    int32_t* accept_len;     // [B]
    int32_t* tokens;         // [B,k+1]
    float* loss;             // [B,k] or null
    void* grad;              // [B,k,V] or null
    float* acc_prob;         // [B,k] or null
    uint32_t* status;        // [B] or null
    // workspace
    uint32_t* ticket;        // [B] zero on entry; reset to zero by the resolver
    uint32_t* wstatus;       // [B] zero on entry; reset to zero by the resolver
    uint8_t* accept;         // [B*k]
    RowConst* rowc;          // [B*(k+1)]
    float* chunk_sums;       // [B*(k+1)*NC]
    int blocks_per_unit;     // blocks that take a ticket per (sequence, row)
};

// ------------------------------------------------------------------------------------------
// element types
template <int DT> struct Elem;
template <> struct Elem<SD_DTYPE_F32> {
    using type = float;
    static constexpr int VEC = 4;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&v)[4]) {
        v[0] = __uint_as_float(q.x); v[1] = __uint_as_float(q.y);
        v[2] = __uint_as_float(q.z); v[3] = __uint_as_float(q.w);
    }
    static __device__ __forceinline__ uint4 pack(const float (&v)[4]) {
        return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]),
                          __float_as_uint(v[3]));
    }
    static __device__ __forceinline__ float load(const void* base, size_t idx) {
        return __ldg(reinterpret_cast<const float*>(base) + idx);
    }
    static __device__ __forceinline__ void store(void* base, size_t idx, float v) {
        reinterpret_cast<float*>(base)[idx] = v;
    }
};
template <> struct Elem<SD_DTYPE_BF16> {
    using type = uint16_t;
    static constexpr int VEC = 8;
    static __device__ __forceinline__ void unpack(const uint4& q, float (&v)[8]) {
        v[0] = __uint_as_float(q.x << 16); v[1] = __uint_as_float(q.x & 0xffff0000u);
        v[2] = __uint_as_float(q.y << 16); v[3] = __uint_as_float(q.y & 0xffff0000u);
        v[4] = __uint_as_float(q.z << 16); v[5] = __uint_as_float(q.z & 0xffff0000u);
        v[6] = __uint_as_float(q.w << 16); v[7] = __uint_as_float(q.w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
        __nv_bfloat162 h = __float22bfloat162_rn(make_float2(lo, hi));
        return *reinterpret_cast<uint32_t*>(&h);
    }
    static __device__ __forceinline__ uint4 pack(const float (&v)[8]) {
        return make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
    }
    static __device__ __forceinline__ float load(const void* base, size_t idx) {
        uint16_t h = __ldg(reinterpret_cast<const uint16_t*>(base) + idx);
        return __uint_as_float(static_cast<uint32_t>(h) << 16);
    }
    static __device__ __forceinline__ void store(void* base, size_t idx, float v) {
        __nv_bfloat16 h = __float2bfloat16_rn(v);
        reinterpret_cast<uint16_t*>(base)[idx] = *reinterpret_cast<uint16_t*>(&h);
    }
};

// ------------------------------------------------------------------------------------------
// scalar helpers
__device__ __forceinline__ float ex2f(float a) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
    return r;
}
__device__ __forceinline__ float neg_ref(float m, float c) { return -__fmul_rn(m, c); }
__device__ __forceinline__ float exp_term(float z, float c, float negR) {
    return ex2f(__fmaf_rn(z, c, negR));
}
// (q-p)/tau of one element of a pair row
__device__ __forceinline__ float grad_elem(float t, float d, float c, const RowConst& rc) {
    float eT = exp_term(t, c, rc.negRT);
    float eD = exp_term(d, c, rc.negRD);
    return __fmaf_rn(eD, rc.kD, -__fmul_rn(eT, rc.kT));
}
// p of one element of a bonus row
__device__ __forceinline__ float prob_elem(float t, float c, const RowConst& rc) {
    return __fmul_rn(exp_term(t, c, rc.negRT), rc.kT);
}

// Per-lane running softmax statistics of a row pair; every lane keeps its own reference.
struct LaneStats {
    float mT, negRT, sT, w;
    float mD, negRD, sD;
    __device__ __forceinline__ void init(float c) {
        mT = mD = -3.402823466e+38f;
        negRT = negRD = fminf(neg_ref(mT, c), 3.402823466e+38f);   // finite, so masked (-inf) entries give 0
        sT = sD = w = 0.f;
    }
    // The KL accumulator w = sum eT*((t-mT)-(d-mD)) is kept relative to both running maxima, so a
    // constant offset between the two models' logits cancels exactly instead of in the last bits.
    // Both maxima move in one step: with identical rows the correction (dT - dD) is exactly zero.
    template <int VEC>
    __device__ __forceinline__ void add_pair(const float (&t)[VEC], const float (&d)[VEC], float c) {
        float vmT = t[0], vmD = d[0];
#pragma unroll
        for (int e = 1; e < VEC; ++e) {
            vmT = fmaxf(vmT, t[e]);
            vmD = fmaxf(vmD, d[e]);
        }
        if (vmT > mT || vmD > mD) {
            const float nT = fmaxf(mT, vmT), nD = fmaxf(mD, vmD);
            const float nrT = (nT > mT) ? neg_ref(nT, c) : negRT;
            const float nrD = (nD > mD) ? neg_ref(nD, c) : negRD;
            const float fT = (nT > mT) ? ex2f(nrT - negRT) : 1.f;
            const float fD = (nD > mD) ? ex2f(nrD - negRD) : 1.f;
            w = (sT > 0.f) ? (w - sT * ((nT - mT) - (nD - mD))) * fT : 0.f;
            sT *= fT;
            sD *= fD;
            mT = nT; negRT = nrT;
            mD = nD; negRD = nrD;
        }
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            float eT = exp_term(t[e], c, negRT);
            float eD = exp_term(d[e], c, negRD);
            sT += eT;
            sD += eD;
            float diff = (t[e] - mT) - (d[e] - mD);
            w = (eT > 0.f) ? __fmaf_rn(eT, diff, w) : w;   // masked target entries (p = 0) add nothing
        }
    }
    template <int VEC>
    __device__ __forceinline__ void add_target(const float (&t)[VEC], float c) {
        float vm = t[0];
#pragma unroll
        for (int e = 1; e < VEC; ++e) vm = fmaxf(vm, t[e]);
        if (vm > mT) {
            float nr = neg_ref(vm, c);
            sT *= ex2f(nr - negRT);
            mT = vm;
            negRT = nr;
        }
    }
    template <int VEC>
    __device__ __forceinline__ void add_bonus(const float (&t)[VEC], float c) {
        add_target<VEC>(t, c);
#pragma unroll
        for (int e = 0; e < VEC; ++e) sT += exp_term(t[e], c, negRT);
    }
};

__device__ __forceinline__ double shfl_xor_f64(double v, int off) {
    return __shfl_xor_sync(0xffffffffu, v, off);
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    return v;
}

// Shared scratch of the block-level reduction of the statistics.
struct StatScratch {
    float wmaxT[kWarps], wmaxD[kWarps];
    double wsT[kWarps], wsD[kWarps], ww[kWarps];
};

// Statistics of everything the block has seen, in every thread.  All threads must call.
// Lanes are first brought to the block's maxima (one fp32 rescale each), then summed in fp64 in
// a fixed order, so the result does not depend on scheduling and costs no serial fp64 exp.
__device__ inline PartialStats block_reduce_stats(const LaneStats& ls, float c, StatScratch& sc) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const float wmT = warp_max_f32(ls.mT), wmD = warp_max_f32(ls.mD);
    if (lane == 0) { sc.wmaxT[warp] = wmT; sc.wmaxD[warp] = wmD; }
    __syncthreads();
    float bmT = sc.wmaxT[0], bmD = sc.wmaxD[0];
#pragma unroll
    for (int w = 1; w < kWarps; ++w) { bmT = fmaxf(bmT, sc.wmaxT[w]); bmD = fmaxf(bmD, sc.wmaxD[w]); }
    float sT = 0.f, wv = 0.f, sD = 0.f;
    if (ls.sT > 0.f) {
        const float f = (ls.mT == bmT) ? 1.f : ex2f(neg_ref(bmT, c) - ls.negRT);
        sT = ls.sT * f;
        wv = (ls.w - ls.sT * ((bmT - ls.mT) - (bmD - ls.mD))) * f;
    }
    if (ls.sD > 0.f) sD = ls.sD * ((ls.mD == bmD) ? 1.f : ex2f(neg_ref(bmD, c) - ls.negRD));
    double dT = (double)sT, dW = (double)wv, dD = (double)sD;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        dT += shfl_xor_f64(dT, off);
        dW += shfl_xor_f64(dW, off);
        dD += shfl_xor_f64(dD, off);
    }
    if (lane == 0) { sc.wsT[warp] = dT; sc.ww[warp] = dW; sc.wsD[warp] = dD; }
    __syncthreads();
    PartialStats r;
    r.mT = bmT; r.mD = bmD;
    r.sT = r.sD = r.w = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { r.sT += sc.wsT[w]; r.w += sc.ww[w]; r.sD += sc.wsD[w]; }
    return r;
}

// Merge of the block statistics of a cluster by one full warp: lane j takes block j, one fp64
// exp2 per lane in parallel, then a butterfly sum.  Every lane returns the row statistics.
__device__ inline PartialStats warp_merge_partials(const PartialStats* p, int n, float c) {
    const int lane = threadIdx.x & 31;
    PartialStats m;
    m.mT = m.mD = -3.402823466e+38f;
    m.sT = m.sD = m.w = 0.0;
    if (lane < n) m = p[lane];
    PartialStats r;
    r.mT = warp_max_f32(m.mT);
    r.mD = warp_max_f32(m.mD);
    double sT = 0.0, wv = 0.0, sD = 0.0;
    if (m.sT > 0.0) {
        const double f = (m.mT == r.mT) ? 1.0 : exp2((double)__fmul_rn(m.mT, c) - (double)__fmul_rn(r.mT, c));
        sT = m.sT * f;
        wv = (m.w - m.sT * (((double)r.mT - (double)m.mT) - ((double)r.mD - (double)m.mD))) * f;
    }
    if (m.sD > 0.0)
        sD = m.sD * ((m.mD == r.mD) ? 1.0 : exp2((double)__fmul_rn(m.mD, c) - (double)__fmul_rn(r.mD, c)));
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        sT += shfl_xor_f64(sT, off);
        wv += shfl_xor_f64(wv, off);
        sD += shfl_xor_f64(sD, off);
    }
    r.sT = sT; r.w = wv; r.sD = sD;
    return r;
}

// ------------------------------------------------------------------------------------------
// block-wide helpers (all threads of the block must call them)
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// Sum over the block in a fixed order; result in every thread.  scratch: kWarps doubles.
__device__ inline double block_sum(double v, double* scratch) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) t += scratch[w];
    return t;
}

// Exclusive prefix sum over the block in thread order; `total` receives the block sum.
__device__ inline double block_exclusive_scan(double v, double* scratch, double* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        double o = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += o;
    }
    __syncthreads();
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    double base = 0.0, tot = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        double s = scratch[w];
        if (w < warp) base += s;
        tot += s;
    }
    *total = tot;
    return base + incl - v;
}

// ------------------------------------------------------------------------------------------
// Constants of a finished row for the second sweep and the inverse-CDF search.
__device__ __forceinline__ RowConst row_constants(const Params& P, bool bonus, const PartialStats& st) {
    RowConst rc;
    rc.negRT = neg_ref(st.mT, P.c);
    rc.negRD = bonus ? 0.f : neg_ref(st.mD, P.c);
    rc.kT = (float)((bonus ? 1.0 : P.inv_tau) / st.sT);
    rc.kD = bonus ? 0.f : (float)(P.inv_tau / st.sD);
    return rc;
}

// What the accept test of one pair row needs from global memory; loaded early by the thread that
// will finish the row so that the latency is off the critical path.
struct AcceptOperands {
    int32_t x;
    float u, tx, dx;
    bool valid;
};
template <int DT>
__device__ __forceinline__ AcceptOperands load_accept_operands(const Params& P, int b, int i) {
    AcceptOperands a;
    a.x = P.x[b * P.k + i];
    a.u = P.u[b * (P.k + 1) + i];
    a.valid = (a.x >= 0 && a.x < P.V);
    a.tx = a.dx = 0.f;
    if (a.valid) {
        a.tx = Elem<DT>::load(P.T, (size_t)(b * (P.k + 1) + i) * P.V + a.x);
        a.dx = Elem<DT>::load(P.D, (size_t)(b * P.k + i) * P.V + a.x);
    }
    return a;
}

// End of a (sequence, row) unit, by one thread: row constants to the workspace, the KL loss and
// the rejection test of the row's draft token.
__device__ inline void finish_row(const Params& P, int b, int i, const PartialStats& st, const RowConst& rc,
                                  const AcceptOperands& op) {
    const bool bonus = (i == P.k);
    const int unit = b * (P.k + 1) + i;
    uint32_t flags = 0;
    const bool okT = (st.sT > 0.0) && isfinite(st.sT);
    const bool okD = bonus || ((st.sD > 0.0) && isfinite(st.sD));
    if (!okT || !okD) flags |= SD_STATUS_BAD_ROW;
    P.rowc[unit] = rc;
    if (!bonus) {
        // log2 of the softmax denominators at temperature tau, reference = the row maximum:
        // the elementwise reference fl(m*c) differs from m*c by eps, which is known exactly.
        const double epsT = (double)st.mT * (double)P.c - (double)__fmul_rn(st.mT, P.c);
        const double epsD = (double)st.mD * (double)P.c - (double)__fmul_rn(st.mD, P.c);
        const double l2ST = log2(st.sT) - epsT;   // log2 sum_v 2^((t_v - mT) c)
        const double l2SD = log2(st.sD) - epsD;
        if (P.loss) {
            // KL(p||q) = ln2 * [ c * E_p((t-mT)-(d-mD)) - log2 S_T + log2 S_D ], S relative to the maxima
            const double kl = 0.6931471805599453 * (P.c64 * (st.w / st.sT) - l2ST + l2SD);
            P.loss[b * P.k + i] = (float)kl;
        }
        // rejection test for draft token x[b,i] with ratio p(x)/q(x) in fp64
        bool acc = false;
        if (!op.valid) {
            flags |= SD_STATUS_BAD_TOKEN;
        } else if (okT && okD) {
            const double tx = (double)op.tx, dx = (double)op.dx;
            double rho;
            if (dx == -INFINITY) {
                rho = (tx == -INFINITY) ? 0.0 : INFINITY;
            } else {
                const double l2p = (tx - (double)st.mT) * P.c64 - l2ST;
                const double l2q = (dx - (double)st.mD) * P.c64 - l2SD;
                rho = exp2(l2p - l2q);
            }
            const double thr = rho < 1.0 ? rho : 1.0;
            acc = (double)op.u < thr;
        }
        P.accept[b * P.k + i] = acc ? 1 : 0;
    }
    if (flags) atomicOr(&P.wstatus[b], flags);
}

// ------------------------------------------------------------------------------------------
// Last block of a sequence: accept length, emitted tokens, the residual / bonus draw.
// Reads what other blocks wrote (after their fence + ticket), so those loads bypass L1.

// Unnormalised mass of vocabulary entry v in the distribution the extra token is drawn from.
//   mode 0: pair row, max(0,p-q)/tau     mode 1: bonus row, p     mode 2: pair row, p/tau
template <int DT>
__device__ __forceinline__ float mass_elem(const Params& P, const RowConst& rc, int mode,
                                           size_t offT, size_t offD, int v) {
    if (v >= P.V) return 0.f;
    const float t = Elem<DT>::load(P.T, offT + v);
    if (mode != 0) return prob_elem(t, P.c, rc);
    const float d = Elem<DT>::load(P.D, offD + v);
    return fmaxf(-grad_elem(t, d, P.c, rc), 0.f);
}

struct ResolveScratch {
    double red[kWarps];
    int found;
    int n;
    int ticket_last;
};

// Inverse-CDF search inside one sampling chunk.  prefix = mass before the chunk, t = target.
// last_with_mass: ignore t and return the last entry of the chunk that has mass.
// Returns the vocabulary index, or -1 if the chunk has no qualifying entry.
template <int DT>
__device__ int search_chunk(const Params& P, const RowConst& rc, int mode, size_t offT, size_t offD,
                            int chunk, double prefix, double t, bool last_with_mass,
                            ResolveScratch& S, double* chunk_total) {
    constexpr int CE = kChunkVecs * Elem<DT>::VEC;
    constexpr int PER = CE / kThreads;            // contiguous entries per thread
    const int tid = threadIdx.x;
    const int v0 = chunk * CE + tid * PER;
    float r[PER];
    double loc = 0.0;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
        r[e] = mass_elem<DT>(P, rc, mode, offT, offD, v0 + e);
        loc += (double)r[e];
    }
    double run = prefix + block_exclusive_scan(loc, S.red, chunk_total);
    if (tid == 0) S.found = last_with_mass ? -1 : 0x7fffffff;
    __syncthreads();
    if (!last_with_mass) {
#pragma unroll
        for (int e = 0; e < PER; ++e) {
            run += (double)r[e];
            if (run > t && r[e] > 0.f) { atomicMin(&S.found, v0 + e); break; }
        }
    } else {
#pragma unroll
        for (int e = 0; e < PER; ++e)
            if (r[e] > 0.f) atomicMax(&S.found, v0 + e);
    }
    __syncthreads();
    const int y = S.found;
    __syncthreads();
    return y == 0x7fffffff ? -1 : y;
}

// Draw from a row without chunk sums (two sweeps over the row by one block).  Only used when a
// rejection leaves no residual mass in fp32, which exact arithmetic rules out.
template <int DT>
__device__ int draw_row_slow(const Params& P, const RowConst& rc, int mode, size_t offT,
                             size_t offD, double u, ResolveScratch& S) {
    double total = 0.0, ctot;
    for (int j = 0; j < P.NC; ++j) {
        search_chunk<DT>(P, rc, mode, offT, offD, j, 0.0, 0.0, true, S, &ctot);
        total += ctot;
    }
    if (!(total > 0.0) || !isfinite(total)) return 0;
    const double t = u * total;
    double prefix = 0.0;
    int last_mass = -1;
    for (int j = 0; j < P.NC; ++j) {
        const int y = search_chunk<DT>(P, rc, mode, offT, offD, j, prefix, t, false, S, &ctot);
        if (y >= 0) return y;
        if (ctot > 0.0) last_mass = j;
        prefix += ctot;
    }
    if (last_mass < 0) return 0;
    const int y = search_chunk<DT>(P, rc, mode, offT, offD, last_mass, 0.0, 0.0, true, S, &ctot);
    return y < 0 ? 0 : y;
}

template <int DT>
__device__ void resolve_sequence(const Params& P, int b, ResolveScratch& S) {
    const int tid = threadIdx.x;
    const int k = P.k, NC = P.NC;

    if (tid == 0) {
        int n = k;
        for (int i = 0; i < k; ++i)
            if (__ldcg(P.accept + b * k + i) == 0) { n = i; break; }
        S.n = n;
    }
    __syncthreads();
    const int n = S.n;
    uint32_t flags = 0;

    // diagnostic: acceptance probability 1 - sum max(0,p-q) per position (Eq. 1)
    if (P.acc_prob) {
        for (int i = 0; i < k; ++i) {
            const float* csi = P.chunk_sums + (size_t)(b * (k + 1) + i) * NC;
            double part = 0.0;
            for (int j = tid; j < NC; j += kThreads) part += (double)__ldcg(csi + j);
            const double R = block_sum(part, S.red) * (double)P.tau;
            if (tid == 0) P.acc_prob[b * k + i] = (float)(1.0 - R);
        }
    }

    const bool bonus = (n == k);
    const int unit = b * (k + 1) + n;
    const float* cs = P.chunk_sums + (size_t)unit * NC;
    const float4 rcv = __ldcg(reinterpret_cast<const float4*>(P.rowc + unit));
    const RowConst rc{rcv.x, rcv.y, rcv.z, rcv.w};
    const size_t offT = (size_t)unit * P.V;
    const size_t offD = (size_t)(b * k + (bonus ? 0 : n)) * P.V;
    const double uk = (double)P.u[b * (k + 1) + k];

    // prefix over the chunk sums: each thread owns a contiguous run of chunks
    const int per = (NC + kThreads - 1) / kThreads;
    const int j0 = min(NC, tid * per), j1 = min(NC, j0 + per);
    double mine = 0.0;
    for (int j = j0; j < j1; ++j) mine += (double)__ldcg(cs + j);
    double total;
    const double before = block_exclusive_scan(mine, S.red, &total);
    const double t = uk * total;

    int y = 0;
    if (!(total > 0.0) || !isfinite(total)) {
        if (bonus) {
            flags |= SD_STATUS_BAD_ROW;
        } else {
            flags |= SD_STATUS_ZERO_RESIDUAL;   // draw from p_n instead
            y = draw_row_slow<DT>(P, rc, 2, offT, offD, uk, S);
        }
    } else {
        if (tid == 0) S.found = 0x7fffffff;
        __syncthreads();
        {
            double run = before;
            for (int j = j0; j < j1; ++j) {
                run += (double)__ldcg(cs + j);
                if (run > t) { atomicMin(&S.found, j); break; }
            }
        }
        __syncthreads();
        int chunk = S.found;
        __syncthreads();
        bool past_end = false;
        if (chunk == 0x7fffffff) {
            // rounding pushed u*R to the total: last chunk that holds mass
            past_end = true;
            if (tid == 0) S.found = -1;
            __syncthreads();
            for (int j = j0; j < j1; ++j)
                if (__ldcg(cs + j) > 0.f) atomicMax(&S.found, j);
            __syncthreads();
            chunk = S.found;
            __syncthreads();
        }
        if (chunk >= 0) {
            double pre_part = 0.0;
            for (int j = tid; j < chunk; j += kThreads) pre_part += (double)__ldcg(cs + j);
            const double prefix = block_sum(pre_part, S.red);
            double ctot;
            y = search_chunk<DT>(P, rc, bonus ? 1 : 0, offT, offD, chunk, prefix, t, past_end, S, &ctot);
            // chunk sum and re-summed entries may disagree in the last bits: last entry with mass
            if (y < 0) y = search_chunk<DT>(P, rc, bonus ? 1 : 0, offT, offD, chunk, 0.0, 0.0, true, S, &ctot);
            if (y < 0) y = 0;
        }
    }

    if (tid == 0) {
        P.accept_len[b] = n;
        const uint32_t st = __ldcg(P.wstatus + b) | flags;
        if (P.status) P.status[b] = st;
        // leave the workspace ready for the next call
        P.wstatus[b] = 0;
        P.ticket[b] = 0;
    }
    for (int i = tid; i <= k; i += kThreads)
        P.tokens[b * (k + 1) + i] = (i < n) ? P.x[b * k + i] : (i == n ? y : -1);
}

// Take a ticket for sequence b; true in every thread of the block that arrives last.
__device__ inline bool take_ticket(const Params& P, int b, int* flag_smem) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const uint32_t total = (uint32_t)(P.k + 1) * (uint32_t)P.blocks_per_unit;
        const uint32_t old = atomicAdd(P.ticket + b, 1u);
        *flag_smem = (old == total - 1);
        __threadfence();
    }
    __syncthreads();
    return *flag_smem != 0;
}

}  // namespace sdv
