// Device-side building blocks of the verify-and-feedback kernels (sm_100a).
//
// Arithmetic contract shared by every kernel in this library, so that a value recomputed later
// (the inverse-CDF search inside a sampling region) is bit-identical to the value summed earlier:
//   c      = fp32(log2(e)/tau)
//   a_v    = fma(z_v, c, -R),  R an INTEGER >= max_v z_v*c  (the reference of the exponentials)
//   e_v    = ex2.approx.ftz(a_v)
//   g_v    = fma(eD_v, kD, -(eT_v*kT)),          kX = fp32((1/tau)/S_X)       [ = (q-p)/tau ]
//   r_v    = max(0, -g_v)                                                      [ = max(0,p-q)/tau ]
//   bonus row: r_v = eT_v * kT with kT = fp32(1/S_T)                           [ = p ]
// Because references are integers, sums taken under different references (by different warps or
// blocks) are brought together by exact multiplications with powers of two: no exponential is
// evaluated outside the elementwise sweeps.  Partial sums are combined in fp64 in a fixed order,
// so results do not depend on scheduling.
#pragma once

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/sd_verify.h"

namespace sdv {

namespace cg = cooperative_groups;

constexpr int kMaxCluster = 8;
constexpr int kMaxLearners = 8;                  // draft models of an online ensemble
constexpr int kGenericRegionElems = 512;         // sampling region of the generic path
constexpr int kRegionRows = 2;                   // fast path: 16-byte vectors per lane and row in a sampling region
constexpr int kRegionVecs = 32 * kRegionRows;    // ... so a region is 64 vectors (1 KiB) of a row
constexpr uint32_t kStatusTimeout = 0x80000000u; // a bounded wait gave up
constexpr uint32_t kWaitLimit = 1u << 21;        // polls of an mbarrier before giving up
constexpr long long kWaitCycles = 2000000000ll;  // ... or about a second of waiting

// Constants a finished row leaves behind for the inverse-CDF search.
struct __align__(16) RowConst {
    float negRT;  // -fl(mT*c)
    float negRD;  // -fl(mD*c)
    float kT;     // pair row: (1/tau)/S_T ; bonus row: 1/S_T
    float kD;     // pair row: (1/tau)/S_D ; bonus row: 0
};

// Softmax statistics of a part of one row pair, relative to integer references RT and RD.
struct __align__(16) PartialStats {
    float RT, RD;      // references of the exponentials (integer values)
    double sT, sD;     // sum of eT = 2^aT, aT = t*c - RT; sum of eD likewise
    double w;          // sum of eT*(aT - aD)
};
// ---- range checks of the checked build ------------------------------------------------------
// With -DSD_BOUNDS_CHECK every index the kernels form into global memory is tested against its
// extent before the access: SD_IN(index, limit, site) is false for an index outside [0, limit), the
// access is then skipped, and the first violation (site, index, limit) and their number are kept
// for sd_bounds_report.  Without the flag SD_IN is the constant true and costs nothing.
#ifdef SD_BOUNDS_CHECK
__device__ unsigned long long g_sd_bounds[4];    // violations; site of the first; its index; its limit
__device__ __noinline__ void sd_bounds_record(long long idx, long long limit, int site) {
    if (atomicAdd(&g_sd_bounds[0], 1ull) == 0ull) {
        g_sd_bounds[1] = (unsigned long long)site;
        g_sd_bounds[2] = (unsigned long long)idx;
        g_sd_bounds[3] = (unsigned long long)limit;
    }
}
__device__ __forceinline__ bool sd_in(long long idx, long long limit, int site) {
    if (idx >= 0 && idx < limit) return true;
    sd_bounds_record(idx, limit, site);
    return false;
}
#define SD_IN(idx, limit, site) (::sdv::sd_in((long long)(idx), (long long)(limit), (site)))
#else
#define SD_IN(idx, limit, site) (true)
#endif
// Sites: 1x fast path (10 target copy, 11 draft copy, 12 gradient store, 13 region mass, 14 second try,
// 15 hint), 2x row report and resolver (20 row constants, 21 loss, 22 accept flag, 23 region masses,
// 24 region searched, 25 tokens), 3x element-wise path, 4x greedy, 5x error-position kernel,
// 6x vocabulary-parallel kernels.

constexpr float kEmptyRef = -1073741824.f;       // reference of a part without a finite entry (-2^30)

struct Params {
    const void* T;           // [B,k+1,V]
    const void* D;           // [B,k,V]
    const int32_t* x;        // [B,k]
    const float* u;          // [B,k+1]
    int B, k, V;
    int RE;                  // vocabulary entries per sampling region (a multiple of 32)
    int NR;                  // sampling regions per row: ceil(V / RE)
    float c;                 // fp32(log2e/tau)
    float tau;
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
    uint32_t* sticky;        // [1] zero on entry; set (and left set) when a bounded wait gave up
    uint8_t* accept;         // [B*k]
    RowConst* rowc;          // [B*(k+1)]
    float* region_sums;      // [B*(k+1)*NR] mass of each sampling region of each row
    int blocks_per_unit;     // blocks that take a ticket per (sequence, row)
    uint32_t wait_polls;     // polls after which a bounded wait gives up (kWaitLimit unless a caller asks otherwise)
    // hint error of the optimistic update (null: not asked for)
    const void* hint;        // [B,k,V] the last round's gradient, in the dtype of the logits
    float* hint_err;         // [B,k] sum_v (hint - this round's gradient)^2
    double* hint_part;       // workspace [B*(k+1)][kMaxCluster]: each block's share of a row's sum
    // online ensemble: feedback of `learners` draft models against one target (0: the plain step).
    // Then loss is [learners,B,k], D and grad above are unused, and nothing is verified or drawn.
    int learners;
    const void* Dn[kMaxLearners];   // [B,k,V] each
    void* Gn[kMaxLearners];         // [B,k,V] each, or null
};

// What a unit of the fast path works on.  Plain step: unit = (sequence, row) with the bonus row
// last.  Ensemble: unit = (sequence, row, learner) with the learner running fastest, so that the
// units that read the same target row follow one another and find it in L2.
struct UnitRef {
    int b, i, n;
    bool bonus;
    size_t t_row;            // row of T
    size_t d_row;            // row of the draft logits and of the gradient (a valid row on a bonus unit too)
};
template <bool ENS>
__device__ __forceinline__ UnitRef unit_ref(const Params& P, int unit) {
    UnitRef r;
    if constexpr (ENS) {
        const int pos = unit / P.learners;
        r.n = unit - pos * P.learners;
        r.b = pos / P.k;
        r.i = pos - r.b * P.k;
        r.bonus = false;
        r.t_row = (size_t)r.b * (P.k + 1) + r.i;
        r.d_row = (size_t)pos;
    } else {
        const int K1 = P.k + 1;
        r.n = 0;
        r.b = unit / K1;
        r.i = unit - r.b * K1;
        r.bonus = (r.i == P.k);
        r.t_row = (size_t)unit;
        r.d_row = (size_t)r.b * P.k + (r.bonus ? 0 : r.i);
    }
    return r;
}
template <bool ENS>
__device__ __forceinline__ int total_units(const Params& P) {
    return ENS ? P.B * P.k * P.learners : P.B * (P.k + 1);
}

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
    static __device__ __forceinline__ uint4 masked() {   // a vector of -inf: adds nothing anywhere
        return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
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
    static __device__ __forceinline__ uint4 masked() {
        return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
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
// Integer reference for exponentials of logits whose maximum is m: ceil(m*c), kept inside
// [-2^30, 2^30] so that it converts to int and differences of references are exact.
__device__ __forceinline__ float ref_of(float m, float c) {
    return fminf(fmaxf(ceilf(__fmul_rn(fmaxf(m, -1e30f), c)), kEmptyRef), 1073741824.f);
}
__device__ __forceinline__ float exp_term(float z, float c, float negR) {
    return ex2f(__fmaf_rn(z, c, negR));
}
// (q-p)/tau of one element of a pair row
__device__ __forceinline__ float grad_elem(float t, float d, float c, const RowConst& rc) {
    float eT = exp_term(t, c, rc.negRT);
    float eD = exp_term(d, c, rc.negRD);
    return __fmaf_rn(eD, rc.kD, -__fmul_rn(eT, rc.kT));
}
// The same for two elements at once (packed fp32 instructions, same rounding).
__device__ __forceinline__ float2 grad_elem2(float2 t, float2 d, float c, const RowConst& rc) {
    const float2 c2 = make_float2(c, c);
    const float2 aT = __ffma2_rn(t, c2, make_float2(rc.negRT, rc.negRT));
    const float2 aD = __ffma2_rn(d, c2, make_float2(rc.negRD, rc.negRD));
    const float2 eT = make_float2(ex2f(aT.x), ex2f(aT.y));
    const float2 eD = make_float2(ex2f(aD.x), ex2f(aD.y));
    const float2 pT = __fmul2_rn(eT, make_float2(-rc.kT, -rc.kT));        // -(eT*kT), exact negation
    return __ffma2_rn(eD, make_float2(rc.kD, rc.kD), pT);
}
// p of one element of a bonus row
__device__ __forceinline__ float prob_elem(float t, float c, const RowConst& rc) {
    return __fmul_rn(exp_term(t, c, rc.negRT), rc.kT);
}
// 2^d as a double for an integer-valued d <= 0; 0 when the result would not be a normal number.
__device__ __forceinline__ double pow2_neg(float d) {
    const int e = (int)fmaxf(d, -2000.f);
    return e < -1022 ? 0.0 : __hiloint2double((1023 + e) << 20, 0);
}

// The same as a float; 0 below the normal range.
__device__ __forceinline__ float pow2_neg_f32(float d) {
    const int e = (int)fmaxf(d, -200.f);
    return e < -126 ? 0.f : __int_as_float((127 + e) << 23);
}

// Sum of VEC values as a balanced tree (short dependency chains, fixed order).
template <int VEC>
__device__ __forceinline__ float tree_sum(const float (&v)[VEC]) {
    if constexpr (VEC == 1) return v[0];
    else if constexpr (VEC == 2) return v[0] + v[1];
    else if constexpr (VEC == 4) return (v[0] + v[1]) + (v[2] + v[3]);
    else return ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
}
// Largest of three (one instruction on sm_100).
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
template <int VEC>
__device__ __forceinline__ float tree_max(const float (&v)[VEC]) {
    if constexpr (VEC == 1) return v[0];
    else if constexpr (VEC == 2) return fmaxf(v[0], v[1]);
    else if constexpr (VEC == 4) return fmaxf(fmax3(v[0], v[1], v[2]), v[3]);
    else return fmax3(fmax3(v[0], v[1], v[2]), fmax3(v[3], v[4], v[5]), fmaxf(v[6], v[7]));
}

// Softmax sums of one lane relative to integer references that the lane's whole warp shares:
//   sT = sum eT, sD = sum eD, w = sum eT*(aT - aD)    with a = fma(z, c, -R), e = ex2(a).
// aT - aD is log2(p/q) up to the two row constants, so w/sT leads to KL(p||q); each a is relative
// to its own row's reference, so an offset between the two models' logits drops out.
struct LaneSums {
    float sT, sD, w;
    __device__ __forceinline__ void init() { sT = sD = w = 0.f; }
    // Move the sums to references larger by dT >= 0 and dD >= 0 (integers): exact.
    __device__ __forceinline__ void rescale(float dT, float dD) {
        const float f = pow2_neg_f32(-dT), g = pow2_neg_f32(-dD);
        w = (sT > 0.f) ? (w - sT * (dT - dD)) * f : 0.f;
        sT *= f;
        sD *= g;
    }
    template <int VEC>
    __device__ __forceinline__ void add_pair(const float (&t)[VEC], const float (&d)[VEC], float c, float negRT,
                                             float negRD) {
        float eT[VEC], eD[VEC], pw[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) {
            const float aT = __fmaf_rn(t[e], c, negRT), aD = __fmaf_rn(d[e], c, negRD);
            eT[e] = ex2f(aT);
            eD[e] = ex2f(aD);
            pw[e] = (eT[e] > 0.f) ? eT[e] * (aT - aD) : 0.f;   // masked target entries (p = 0) add nothing
        }
        sT += tree_sum<VEC>(eT);
        sD += tree_sum<VEC>(eD);
        w += tree_sum<VEC>(pw);
    }
    // The same for one vector, into partial sums of its own (short dependency chains).  Entries are
    // taken two at a time with the packed fp32 instructions of sm_100 (same rounding as the scalar
    // ones); even and odd entries are summed separately and meet at the end.
    // MASKED = false leaves out the test for masked target entries (p = 0 exactly, logit -inf):
    // there eT = 0 meets aT - aD = -inf or NaN and the product is NaN instead of 0, so the caller
    // must look at pW and do the vector again with MASKED = true when it is NaN.  It saves three
    // of thirteen instructions per two entries on rows without masked entries, which is most rows.
    template <int VEC, bool MASKED = true>
    static __device__ __forceinline__ void vector_pair(const float (&t)[VEC], const float (&d)[VEC], float c,
                                                       float negRT, float negRD, float& pT, float& pD, float& pW) {
        static_assert(VEC % 2 == 0, "packed arithmetic takes entries in pairs");
        const float2 c2 = make_float2(c, c), nT2 = make_float2(negRT, negRT), nD2 = make_float2(negRD, negRD);
        const float2 m1 = make_float2(-1.f, -1.f);
        float2 accT = make_float2(0.f, 0.f), accD = make_float2(0.f, 0.f), accW = make_float2(0.f, 0.f);
#pragma unroll
        for (int e = 0; e < VEC; e += 2) {
            const float2 aT = __ffma2_rn(make_float2(t[e], t[e + 1]), c2, nT2);
            const float2 aD = __ffma2_rn(make_float2(d[e], d[e + 1]), c2, nD2);
            const float2 eT = make_float2(ex2f(aT.x), ex2f(aT.y));
            const float2 eD = make_float2(ex2f(aD.x), ex2f(aD.y));
            const float2 diff = __ffma2_rn(aD, m1, aT);          // aT - aD
            if constexpr (MASKED) {
                if (eT.x > 0.f) accW.x = __fmaf_rn(eT.x, diff.x, accW.x);    // masked target entries (p = 0) add nothing
                if (eT.y > 0.f) accW.y = __fmaf_rn(eT.y, diff.y, accW.y);
            } else {
                accW = __ffma2_rn(eT, diff, accW);               // same products, same order, same rounding
            }
            accT = __fadd2_rn(accT, eT);
            accD = __fadd2_rn(accD, eD);
        }
        pT = accT.x + accT.y;
        pD = accD.x + accD.y;
        pW = accW.x + accW.y;
    }
    template <int VEC>
    static __device__ __forceinline__ float vector_bonus(const float (&t)[VEC], float c, float negRT) {
        float eT[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) eT[e] = exp_term(t[e], c, negRT);
        return tree_sum<VEC>(eT);
    }
    template <int VEC>
    __device__ __forceinline__ void add_bonus(const float (&t)[VEC], float c, float negRT) {
        float eT[VEC];
#pragma unroll
        for (int e = 0; e < VEC; ++e) eT[e] = exp_term(t[e], c, negRT);
        sT += tree_sum<VEC>(eT);
    }
};

// ------------------------------------------------------------------------------------------
// warp-wide helpers (all 32 lanes of the warp must call them)
__device__ __forceinline__ double shfl_xor_f64(double v, int off) {
    return __shfl_xor_sync(0xffffffffu, v, off);
}
__device__ __forceinline__ float warp_max_f32(float v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, off));
    return v;
}
// Largest of the lanes' integer-valued references (one redux instruction).
__device__ __forceinline__ float warp_max_ref(float R) {
    return (float)__reduce_max_sync(0xffffffffu, (int)R);
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}
// Inclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ double warp_inclusive_scan(double v) {
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        double o = __shfl_up_sync(0xffffffffu, v, off);
        if (lane >= off) v += o;
    }
    return v;
}

// A partial rescaled from its own references to (RT, RD); exact, because references are integers.
__device__ __forceinline__ PartialStats rescaled(const PartialStats& m, float RT, float RD) {
    PartialStats r;
    r.RT = RT; r.RD = RD;
    const double f = pow2_neg(m.RT - RT), g = pow2_neg(m.RD - RD);
    r.sT = m.sT * f;
    r.sD = m.sD * g;
    r.w = (m.sT > 0.0 && f > 0.0) ? (m.w - m.sT * (double)((RT - m.RT) - (RD - m.RD))) * f : 0.0;
    return r;
}
__device__ __forceinline__ PartialStats empty_partial() {
    PartialStats m;
    m.RT = m.RD = kEmptyRef;
    m.sT = m.sD = m.w = 0.0;
    return m;
}

// Merge of up to 16 partials in shared memory by every calling lane on its own, in index order:
// no lane talks to another, and all lanes get the same bits.
__device__ __forceinline__ PartialStats merge_partials_serial(const PartialStats* p, int n) {
    float RT = kEmptyRef, RD = kEmptyRef;
    for (int i = 0; i < n; ++i) { RT = fmaxf(RT, p[i].RT); RD = fmaxf(RD, p[i].RD); }
    PartialStats r;
    r.RT = RT; r.RD = RD;
    r.sT = r.sD = r.w = 0.0;
    for (int i = 0; i < n; ++i) {
        const PartialStats q = rescaled(p[i], RT, RD);
        r.sT += q.sT; r.sD += q.sD; r.w += q.w;
    }
    return r;
}

// Merge of 32 partials, one per lane (lanes without one pass empty_partial()), by the whole warp:
// largest references by one redux each, exact rescaling, butterfly sums in a fixed order.  Every
// lane gets the same bits.
__device__ __forceinline__ PartialStats warp_merge_lanes(const PartialStats& m) {
    const float RT = warp_max_ref(m.RT), RD = warp_max_ref(m.RD);
    PartialStats r = rescaled(m, RT, RD);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        r.sT += shfl_xor_f64(r.sT, off);
        r.sD += shfl_xor_f64(r.sD, off);
        r.w += shfl_xor_f64(r.w, off);
    }
    return r;
}

// Sums of the lanes of a warp that share the references (RT, RD), as one partial in every lane.
__device__ __forceinline__ PartialStats warp_sum_lanes(const LaneSums& ls, float RT, float RD) {
    double dT = (double)ls.sT, dW = (double)ls.w, dD = (double)ls.sD;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        dT += shfl_xor_f64(dT, off);
        dW += shfl_xor_f64(dW, off);
        dD += shfl_xor_f64(dD, off);
    }
    PartialStats r;
    r.RT = RT; r.RD = RD;
    r.sT = dT; r.sD = dD; r.w = dW;
    return r;
}

// ------------------------------------------------------------------------------------------
// Constants of a finished row for the second sweep and the inverse-CDF search.
__device__ __forceinline__ RowConst row_constants_of(double inv_tau, bool bonus, const PartialStats& st) {
    RowConst rc;
    rc.negRT = -st.RT;
    rc.negRD = bonus ? 0.f : -st.RD;
    rc.kT = (float)((bonus ? 1.0 : inv_tau) / st.sT);
    rc.kD = bonus ? 0.f : (float)(inv_tau / st.sD);
    return rc;
}
__device__ __forceinline__ RowConst row_constants(const Params& P, bool bonus, const PartialStats& st) {
    return row_constants_of(P.inv_tau, bonus, st);
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
    if (SD_IN(unit, P.B * (P.k + 1), 20)) P.rowc[unit] = rc;
    if (!bonus) {
        // log2 p_v = aT_v - log2 S_T and log2 q_v = aD_v - log2 S_D, so
        // KL(p||q) = ln2 * [ E_p(aT - aD) - log2 S_T + log2 S_D ]
        const double l2ST = log2(st.sT), l2SD = log2(st.sD);
        if (P.loss && SD_IN(b * P.k + i, P.B * P.k, 21)) {
            const double kl = 0.6931471805599453 * (st.w / st.sT - l2ST + l2SD);
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
                const double l2p = (tx * (double)P.c - (double)st.RT) - l2ST;
                const double l2q = (dx * (double)P.c - (double)st.RD) - l2SD;
                rho = exp2(l2p - l2q);
            }
            const double thr = rho < 1.0 ? rho : 1.0;
            acc = (double)op.u < thr;
        }
        if (SD_IN(b * P.k + i, P.B * P.k, 22)) P.accept[b * P.k + i] = acc ? 1 : 0;
    }
    if (flags) atomicOr(&P.wstatus[b], flags);
}

// End of a (sequence, row, learner) unit of the ensemble feedback, by one thread: the learner's loss.
__device__ inline void finish_row_ensemble(const Params& P, const UnitRef& ur, const PartialStats& st) {
    const bool ok = (st.sT > 0.0) && isfinite(st.sT) && (st.sD > 0.0) && isfinite(st.sD);
    if (!ok && P.status) atomicOr(&P.status[ur.b], SD_STATUS_BAD_ROW);
    const double kl = 0.6931471805599453 * (st.w / st.sT - log2(st.sT) + log2(st.sD));
    P.loss[(size_t)ur.n * P.B * P.k + ur.d_row] = (float)kl;
}

// ------------------------------------------------------------------------------------------
// Resolution of a sequence by one warp, once every (row, slice) of the sequence has been
// processed: accept length, emitted tokens, the residual / bonus draw.  It reads what other
// blocks wrote (after their fence + ticket), so those loads bypass L1.

// Unnormalised mass of a vocabulary entry with target logit t and draft logit d in the distribution
// the extra token is drawn from.
//   mode 0: pair row, max(0,p-q)/tau     mode 1: bonus row, p     mode 2: pair row, p/tau
__device__ __forceinline__ float mass_of(float t, float d, float c, const RowConst& rc, int mode) {
    if (mode != 0) return prob_elem(t, c, rc);
    return fmaxf(-grad_elem(t, d, c, rc), 0.f);
}

// Masses of the PER consecutive entries from v0 on (this lane's share of a sampling region), with
// every load in flight before the first is used: the warp that draws is on the critical path of
// its sequence, and one round trip to L2 is all it should pay per region.  VECTOR: rows are whole
// 16-byte vectors and PER is a multiple of the entries of a vector (fast path); otherwise element
// loads.  Entries past the end of the row have mass 0.
template <int DT, int PER, bool VECTOR>
__device__ __forceinline__ void lane_masses(const Params& P, const RowConst& rc, int mode, size_t offT, size_t offD,
                                            int v0, float (&m)[PER]) {
    using E = Elem<DT>;
    using ET = typename E::type;
    float t[PER], d[PER];
    if constexpr (VECTOR) {
        constexpr int VEC = E::VEC;
        static_assert(PER % VEC == 0, "a lane's share is whole vectors");
        const uint4* pT = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.T) + offT + v0);
        const uint4* pD = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.D) + offD + v0);
        uint4 qt[PER / VEC], qd[PER / VEC];
#pragma unroll
        for (int g = 0; g < PER / VEC; ++g) {
            const bool in = v0 + g * VEC < P.V && SD_IN(v0 + g * VEC + VEC - 1, P.V, 24);
            qt[g] = in ? __ldg(pT + g) : E::masked();
            qd[g] = (in && mode == 0) ? __ldg(pD + g) : E::masked();
        }
#pragma unroll
        for (int g = 0; g < PER / VEC; ++g) {
            float a[VEC], b[VEC];
            E::unpack(qt[g], a);
            E::unpack(qd[g], b);
#pragma unroll
            for (int e = 0; e < VEC; ++e) { t[g * VEC + e] = a[e]; d[g * VEC + e] = b[e]; }
        }
    } else {
#pragma unroll
        for (int e = 0; e < PER; ++e) {
            const bool in = v0 + e < P.V;
            t[e] = in ? E::load(P.T, offT + v0 + e) : -INFINITY;
            d[e] = (in && mode == 0) ? E::load(P.D, offD + v0 + e) : -INFINITY;
        }
    }
#pragma unroll
    for (int e = 0; e < PER; ++e) m[e] = (v0 + e < P.V) ? mass_of(t[e], d[e], P.c, rc, mode) : 0.f;
}

// Inverse-CDF search inside one sampling region.  prefix = mass before the region, t = target.
// last_with_mass: ignore t and return the last entry of the region that has mass.
// Every lane takes a contiguous run of PER = RE/32 entries.  Returns (in every lane) the
// vocabulary index, or -1 if the region has no qualifying entry.
template <int DT, int PER, bool VECTOR>
__device__ int search_region(const Params& P, const RowConst& rc, int mode, size_t offT, size_t offD,
                             int region, double prefix, double t, bool last_with_mass, double* region_total) {
    const int lane = threadIdx.x & 31;
    const int v0 = region * (32 * PER) + lane * PER;
    float m[PER];
    lane_masses<DT, PER, VECTOR>(P, rc, mode, offT, offD, v0, m);
    double loc = 0.0;
#pragma unroll
    for (int e = 0; e < PER; ++e) loc += (double)m[e];
    const double incl = warp_inclusive_scan(loc);
    *region_total = __shfl_sync(0xffffffffu, incl, 31);
    int cand = last_with_mass ? -1 : 0x7fffffff;
    if (!last_with_mass) {
        double run = prefix + (incl - loc);
        if (run + loc > t) {                      // the crossing can only be in a lane whose run reaches t
#pragma unroll
            for (int e = 0; e < PER; ++e) {
                run += (double)m[e];
                if (cand == 0x7fffffff && run > t && m[e] > 0.f) cand = v0 + e;
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) cand = min(cand, __shfl_xor_sync(0xffffffffu, cand, off));
        return cand == 0x7fffffff ? -1 : cand;
    }
    if (loc > 0.0) {
#pragma unroll
        for (int e = 0; e < PER; ++e)
            if (m[e] > 0.f) cand = v0 + e;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) cand = max(cand, __shfl_xor_sync(0xffffffffu, cand, off));
    return cand;
}

// Draw from a row without region sums (two sweeps over the row by one warp).  Only used when a
// rejection leaves no residual mass in fp32, which exact arithmetic rules out.
template <int DT, int PER, bool VECTOR>
__device__ int draw_row_slow(const Params& P, const RowConst& rc, int mode, size_t offT,
                             size_t offD, double u) {
    double total = 0.0, rtot;
    for (int j = 0; j < P.NR; ++j) {
        search_region<DT, PER, VECTOR>(P, rc, mode, offT, offD, j, 0.0, 0.0, true, &rtot);
        total += rtot;
    }
    if (!(total > 0.0) || !isfinite(total)) return 0;
    const double t = u * total;
    double prefix = 0.0;
    int last_mass = -1;
    for (int j = 0; j < P.NR; ++j) {
        const int y = search_region<DT, PER, VECTOR>(P, rc, mode, offT, offD, j, prefix, t, false, &rtot);
        if (y >= 0) return y;
        if (rtot > 0.0) last_mass = j;
        prefix += rtot;
    }
    if (last_mass < 0) return 0;
    const int y = search_region<DT, PER, VECTOR>(P, rc, mode, offT, offD, last_mass, 0.0, 0.0, true, &rtot);
    return y < 0 ? 0 : y;
}

// FAST: the regions are those of the fast path (kRegionVecs vectors, rows of whole vectors);
// otherwise those of the generic path (kGenericRegionElems entries, any alignment).
template <int DT, bool FAST>
__device__ __noinline__ void resolve_sequence(const Params& P, int b) {
    constexpr int PER = FAST ? kRegionVecs * Elem<DT>::VEC / 32 : kGenericRegionElems / 32;
    const int lane = threadIdx.x & 31;
    const int k = P.k, NR = P.NR;

    // The warp that resolves a sequence is the last thing between the kernel and its end, and almost
    // all of its time is memory round trips: everything that does not depend on the accept length is
    // asked for here, in one go, together with the rejection flags.
    const float uk_f = P.u[b * (k + 1) + k];
    const int32_t x_first = (lane < k) ? P.x[b * k + lane] : -1;
    uint32_t st_word = 0, sticky_word = 0;
    if (lane == 0) {
        st_word = __ldcg(P.wstatus + b);
        sticky_word = __ldcg(P.sticky);
    }

    // accept length: first rejected position
    int n = k;
    for (int i0 = 0; i0 < k; i0 += 32) {
        const int i = i0 + lane;
        const bool rej = (i < k) && (__ldcg(P.accept + b * k + i) == 0);
        const unsigned m = __ballot_sync(0xffffffffu, rej);
        if (m) { n = i0 + __ffs(m) - 1; break; }
    }
    uint32_t flags = 0;

    // hint error per position: the shares of the blocks that worked on the row, in their order
    if (P.hint_err) {
        for (int i = lane; i < k; i += 32) {
            const double* hp = P.hint_part + (size_t)(b * (k + 1) + i) * kMaxCluster;
            double e = 0.0;
            for (int r = 0; r < P.blocks_per_unit; ++r) e += __ldcg(hp + r);
            P.hint_err[b * k + i] = (float)e;
        }
    }

    // diagnostic: acceptance probability 1 - sum max(0,p-q) per position (Eq. 1)
    if (P.acc_prob) {
        for (int i = 0; i < k; ++i) {
            const float* rsi = P.region_sums + (size_t)(b * (k + 1) + i) * NR;
            double part = 0.0;
            for (int j = lane; j < NR; j += 32 * 4) {
                float v[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) v[q] = (j + 32 * q < NR) ? __ldcg(rsi + j + 32 * q) : 0.f;
#pragma unroll
                for (int q = 0; q < 4; ++q) part += (double)v[q];
            }
            const double R = warp_sum(part) * (double)P.tau;
            if (lane == 0) P.acc_prob[b * k + i] = (float)(1.0 - R);
        }
    }

    const bool bonus = (n == k);
    const int unit = b * (k + 1) + n;
    if (!SD_IN(unit, P.B * (k + 1), 23) || !SD_IN(n, k + 1, 23)) return;
    const float* rs = P.region_sums + (size_t)unit * NR;
    const float4 rcv = __ldcg(reinterpret_cast<const float4*>(P.rowc + unit));
    const RowConst rc{rcv.x, rcv.y, rcv.z, rcv.w};
    const size_t offT = (size_t)unit * P.V;
    const size_t offD = (size_t)(b * k + (bonus ? 0 : n)) * P.V;
    const double uk = (double)uk_f;

    // prefix over the region sums: each lane owns a contiguous run of regions, which it reads sixteen
    // at a time (all sixteen loads in flight together) and adds up in index order; the first sixteen
    // stay in registers for the search below
    constexpr int kHeld = 16;
    const int per = (NR + 31) / 32;
    const int j0 = min(NR, lane * per), j1 = min(NR, j0 + per);
    float held[kHeld];
#pragma unroll
    for (int q = 0; q < kHeld; ++q) held[q] = (j0 + q < j1) ? __ldcg(rs + j0 + q) : 0.f;
    double mine = 0.0;
#pragma unroll
    for (int q = 0; q < kHeld; ++q) mine += (double)held[q];
    for (int c = j0 + kHeld; c < j1; c += kHeld) {
        float v[kHeld];
#pragma unroll
        for (int q = 0; q < kHeld; ++q) v[q] = (c + q < j1) ? __ldcg(rs + c + q) : 0.f;
#pragma unroll
        for (int q = 0; q < kHeld; ++q) mine += (double)v[q];
    }
    const double incl = warp_inclusive_scan(mine);
    const double before = incl - mine;
    const double total = __shfl_sync(0xffffffffu, incl, 31);
    const double t = uk * total;

    int y = 0;
    if (!(total > 0.0) || !isfinite(total)) {
        if (bonus) {
            flags |= SD_STATUS_BAD_ROW;
        } else {
            flags |= SD_STATUS_ZERO_RESIDUAL;   // draw from p_n instead
            y = draw_row_slow<DT, PER, FAST>(P, rc, 2, offT, offD, uk);
        }
    } else {
        // first region whose running sum exceeds t, and the mass before it
        int cand = 0x7fffffff;
        double cand_prefix = 0.0;
        if (before + mine > t) {                  // the crossing can only be in a lane whose run reaches t
            double run = before;
#pragma unroll
            for (int q = 0; q < kHeld; ++q) {
                if (cand == 0x7fffffff && j0 + q < j1) {
                    const double next = run + (double)held[q];
                    if (next > t) { cand = j0 + q; cand_prefix = run; }
                    else run = next;
                }
            }
            for (int c = j0 + kHeld; c < j1 && cand == 0x7fffffff; c += kHeld) {
                float v[kHeld];
#pragma unroll
                for (int q = 0; q < kHeld; ++q) v[q] = (c + q < j1) ? __ldcg(rs + c + q) : 0.f;
#pragma unroll
                for (int q = 0; q < kHeld; ++q) {
                    if (cand == 0x7fffffff && c + q < j1) {
                        const double next = run + (double)v[q];
                        if (next > t) { cand = c + q; cand_prefix = run; }
                        else run = next;
                    }
                }
            }
        }
        const unsigned has = __ballot_sync(0xffffffffu, cand != 0x7fffffff);
        int region = -1;
        double prefix = 0.0;
        bool past_end = false;
        if (has) {
            const int owner = __ffs(has) - 1;
            region = __shfl_sync(0xffffffffu, cand, owner);
            prefix = __shfl_sync(0xffffffffu, cand_prefix, owner);
        } else {
            // rounding pushed u*R to the total: last region that holds mass
            past_end = true;
            int lastr = -1;
            for (int j = j0; j < j1; ++j)
                if (__ldcg(rs + j) > 0.f) lastr = j;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) lastr = max(lastr, __shfl_xor_sync(0xffffffffu, lastr, off));
            region = lastr;
        }
        if (region >= 0 && SD_IN(region, NR, 24)) {
            double rtot;
            y = search_region<DT, PER, FAST>(P, rc, bonus ? 1 : 0, offT, offD, region, prefix, t, past_end, &rtot);
            // region sum and re-summed entries may disagree in the last bits: last entry with mass
            if (y < 0) y = search_region<DT, PER, FAST>(P, rc, bonus ? 1 : 0, offT, offD, region, 0.0, 0.0, true, &rtot);
            if (y < 0) y = 0;
        }
    }

    if (lane == 0) {
        P.accept_len[b] = n;
        uint32_t st = st_word | flags;
        if (sticky_word != 0) st |= kStatusTimeout;
        if (P.status && st) atomicOr(P.status + b, st);   // zero on entry; a block that gave up may have set its bit already
        // leave the workspace ready for the next call
        P.wstatus[b] = 0;
        P.ticket[b] = 0;
    }
    for (int i = lane; i <= k; i += 32) {
        const int32_t xi = (i == lane) ? x_first : ((i < k) ? P.x[b * k + i] : -1);
        if (SD_IN(b * (k + 1) + i, P.B * (k + 1), 25)) P.tokens[b * (k + 1) + i] = (i < n) ? xi : (i == n ? y : -1);
    }
}

// Tickets of one block for sequence b: `n` of the (k+1) * blocks_per_unit tickets of the
// sequence at once, by one thread, after everything the tickets stand for has been ordered before
// this thread.  True if these were the last tickets of the sequence.
__device__ __forceinline__ bool take_tickets(const Params& P, int b, uint32_t n) {
    __threadfence();
    const uint32_t total = (uint32_t)(P.k + 1) * (uint32_t)P.blocks_per_unit;
    const uint32_t old = atomicAdd(P.ticket + b, n);
    const bool last = (old + n == total);
    if (last) __threadfence();
    return last;
}

}  // namespace sdv
