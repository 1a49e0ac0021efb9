// The step for logits that are sharded along the vocabulary, as a tensor-parallel output layer
// leaves them (the paper's deployment spreads a model over four GPUs): rank g of G holds the
// columns [v_offset, v_offset + Vs) of every logit row.  A softmax needs every column, so the
// step falls into three local phases with two small exchanges between them:
//
//   phase 1  sd_vp_stats_kernel   per row: softmax sums of the shard relative to integer
//                                 references (a PartialStats), and the logits of the drafted
//                                 token if this shard holds it              -> 48 bytes per row
//   exchange all-gather of the records of all ranks
//   phase 2  sd_vp_rows_kernel    per sequence: the G records of every row merged in rank order
//                                 (exact powers of two, fp64 sums: every rank gets the same bits),
//                                 row constants, KL loss, rejection tests, accept length
//            sd_vp_grad_kernel    second sweep over the shard: the gradient's columns of every
//                                 row, and the masses of the sampling regions of the one row per
//                                 sequence that the extra token is drawn from
//            sd_vp_mass_kernel    per sequence: this shard's share of that row's mass, and of the mass
//                                 of p_n (the fallback of a residual without mass)        -> 16 bytes
//   exchange all-gather of the shares
//   phase 3  sd_vp_draw_kernel    per sequence: exclusive scan of the shares in rank order; the rank
//                                 whose interval holds u_k * total searches its own regions and
//                                 writes the token (global index), the others write -1
//   exchange element-wise maximum of the token arrays (the caller's all-reduce)
//
// The arithmetic is that of the single-GPU kernels (same element functions, same merging), so the
// results meet the same bars against the oracle.  Each logit is read from HBM twice here: the
// exchange between the passes is a round trip through the host's collective, and a shard's batch
// does not stay in L2 meanwhile.
#pragma once

#include "sd_kernels.cuh"

namespace sdv {

constexpr int kVpThreads = 256;
constexpr int kVpWarps = kVpThreads / 32;

// What a rank tells the others about its shard of one row.
struct __align__(16) VpRecord {
    PartialStats st;         // 32 bytes
    float tx, dx;            // logits of the drafted token (target, draft) if this shard holds it
    uint32_t has_token;      // 1 if it does
    uint32_t pad;
};
static_assert(sizeof(VpRecord) == 48, "record layout is part of the ABI");

struct VpParams {
    const void* T;           // [B,k+1,Vs]
    const void* D;           // [B,k,Vs]
    const int32_t* x;        // [B,k] global token ids
    const float* u;          // [B,k+1]
    int B, k, Vs, v_offset, V_total;
    int G, rank;
    float c, tau;
    double inv_tau;
    int NR;                  // sampling regions per shard row (kRegionVecs vectors each)
    VpRecord* records;       // phase 1 out: [B*(k+1)]
    const VpRecord* all;     // phase 2 in: [G][B*(k+1)]
    int32_t* accept_len;     // [B]
    float* loss;             // [B,k] or null
    void* grad;              // [B,k,Vs] or null
    uint32_t* status;        // [B] or null
    double* local_mass;      // [B][2]: share of the residual (or bonus) mass, share of the mass of p_n
    const double* all_mass;  // phase 3 in: [G][B][2]
    int32_t* tokens;         // [B,k+1]
    // workspace
    RowConst* rowc;          // [B*(k+1)]
    float* region_sums;      // [B][2][NR]: regions of the row the extra token is drawn from: masses of the
                             // residual (or bonus row), and of p_n (what a residual without mass falls back to)
};

// ---- phase 1 -------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kVpThreads) sd_vp_stats_kernel(const VpParams P) {
    using E = Elem<DT>;
    using ET = typename E::type;
    constexpr int VEC = E::VEC;
    __shared__ PartialStats warp_part[kVpWarps];
    const int unit = blockIdx.x;
    const int K1 = P.k + 1;
    const int b = unit / K1, i = unit - b * K1;
    const bool bonus = (i == P.k);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (!SD_IN(unit, P.B * K1, 60)) return;
    const uint4* Trow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.T) + (size_t)unit * P.Vs);
    const uint4* Drow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.D) + (size_t)(b * P.k + (bonus ? 0 : i)) * P.Vs);
    const int NV = P.Vs / VEC;

    // Two vectors of each row per thread and turn; every turn raises the warp's references to the
    // maxima it has seen (the sums follow by exact powers of two) before it adds.
    float RT = kEmptyRef, RD = kEmptyRef;
    LaneSums ls;
    ls.init();
    for (int v0 = 0; v0 < NV; v0 += 2 * kVpThreads) {
        uint4 qt[2], qd[2];
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            const int vi = v0 + g * kVpThreads + tid;
            qt[g] = vi < NV ? __ldcs(Trow + vi) : E::masked();
            qd[g] = (!bonus && vi < NV) ? __ldcs(Drow + vi) : E::masked();
        }
        float tv[2][VEC], dv[2][VEC];
        float mt = -INFINITY, md = -INFINITY;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            E::unpack(qt[g], tv[g]);
            E::unpack(qd[g], dv[g]);
            mt = fmaxf(mt, tree_max<VEC>(tv[g]));
            md = fmaxf(md, tree_max<VEC>(dv[g]));
        }
        const float nT = fmaxf(RT, warp_max_ref(ref_of(mt, P.c)));
        const float nD = bonus ? kEmptyRef : fmaxf(RD, warp_max_ref(ref_of(md, P.c)));
        ls.rescale(nT - RT, nD - RD);
        RT = nT;
        RD = nD;
#pragma unroll
        for (int g = 0; g < 2; ++g) {
            if (!bonus) {
                float pT, pD, pW;
                LaneSums::vector_pair<VEC, true>(tv[g], dv[g], P.c, -RT, -RD, pT, pD, pW);
                ls.sT += pT;
                ls.sD += pD;
                ls.w += pW;
            } else {
                ls.sT += LaneSums::vector_bonus<VEC>(tv[g], P.c, -RT);
            }
        }
    }
    const PartialStats part = warp_sum_lanes(ls, RT, RD);
    if (lane == 0) warp_part[warp] = part;
    __syncthreads();
    if (tid == 0) {
        VpRecord r;
        r.st = merge_partials_serial(warp_part, kVpWarps);
        r.tx = r.dx = 0.f;
        r.has_token = 0;
        r.pad = 0;
        if (!bonus) {
            const int xg = P.x[b * P.k + i] - P.v_offset;
            if (xg >= 0 && xg < P.Vs) {
                r.has_token = 1;
                r.tx = E::load(P.T, (size_t)unit * P.Vs + xg);
                r.dx = E::load(P.D, (size_t)(b * P.k + i) * P.Vs + xg);
            }
        }
        P.records[unit] = r;
    }
}

// ---- phase 2 -------------------------------------------------------------------------------
// One block per sequence, one thread per row: merge of the G records of the row in rank order,
// row constants, loss, rejection test; then the accept length.  Every rank computes the same bits.
__global__ void __launch_bounds__(96) sd_vp_rows_kernel(const VpParams P) {
    __shared__ int accepted[SD_MAX_K + 1];
    __shared__ uint32_t flags_sh;
    const int b = blockIdx.x, i = threadIdx.x;
    const int K1 = P.k + 1;
    if (i == 0) flags_sh = 0;
    __syncthreads();
    if (i < K1) {
        const int unit = b * K1 + i;
        const bool bonus = (i == P.k);
        const size_t rows = (size_t)P.B * K1;
        float RT = kEmptyRef, RD = kEmptyRef;
        for (int g = 0; g < P.G; ++g) {
            RT = fmaxf(RT, P.all[(size_t)g * rows + unit].st.RT);
            RD = fmaxf(RD, P.all[(size_t)g * rows + unit].st.RD);
        }
        PartialStats st;
        st.RT = RT; st.RD = RD;
        st.sT = st.sD = st.w = 0.0;
        float tx = 0.f, dx = 0.f;
        bool have = false;
        for (int g = 0; g < P.G; ++g) {
            const VpRecord r = P.all[(size_t)g * rows + unit];
            const PartialStats q = rescaled(r.st, RT, RD);
            st.sT += q.sT; st.sD += q.sD; st.w += q.w;
            if (r.has_token && !have) { have = true; tx = r.tx; dx = r.dx; }
        }
        const RowConst rc = row_constants_of(P.inv_tau, bonus, st);
        P.rowc[unit] = rc;
        uint32_t flags = 0;
        const bool okT = (st.sT > 0.0) && isfinite(st.sT);
        const bool okD = bonus || ((st.sD > 0.0) && isfinite(st.sD));
        if (!okT || !okD) flags |= SD_STATUS_BAD_ROW;
        bool acc = true;
        if (!bonus) {
            const double l2ST = log2(st.sT), l2SD = log2(st.sD);
            if (P.loss) P.loss[b * P.k + i] = (float)(0.6931471805599453 * (st.w / st.sT - l2ST + l2SD));
            acc = false;
            const int xg = P.x[b * P.k + i];
            if (xg < 0 || xg >= P.V_total || !have) {
                flags |= SD_STATUS_BAD_TOKEN;
            } else if (okT && okD) {
                const double dtx = (double)tx, ddx = (double)dx;
                double rho;
                if (ddx == -INFINITY) {
                    rho = (dtx == -INFINITY) ? 0.0 : INFINITY;
                } else {
                    const double l2p = (dtx * (double)P.c - (double)st.RT) - l2ST;
                    const double l2q = (ddx * (double)P.c - (double)st.RD) - l2SD;
                    rho = exp2(l2p - l2q);
                }
                acc = (double)P.u[b * K1 + i] < (rho < 1.0 ? rho : 1.0);
            }
        }
        accepted[i] = acc ? 1 : 0;
        if (flags) atomicOr(&flags_sh, flags);
    }
    __syncthreads();
    if (i == 0) {
        int n = P.k;
        for (int j = 0; j < P.k; ++j)
            if (!accepted[j]) { n = j; break; }
        P.accept_len[b] = n;
        if (P.status) P.status[b] = flags_sh;
    }
}

// Second sweep over the shard: one block per (row, slice of sampling regions).  Gradient of every
// pair row; masses of the regions of row n_b of every sequence (the bonus row when n_b = k).
constexpr int kVpSliceRegions = 32;
template <int DT>
__global__ void __launch_bounds__(kVpThreads, 4) sd_vp_grad_kernel(const VpParams P, const int slices) {
    using E = Elem<DT>;
    using ET = typename E::type;
    constexpr int VEC = E::VEC;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int unit = (int)blockIdx.x / slices, sl = (int)blockIdx.x - unit * slices;
    const int K1 = P.k + 1;
    const int b = unit / K1, i = unit - b * K1;
    const bool bonus = (i == P.k);
    const int n = P.accept_len[b];
    const bool draws = (i == n);                     // the extra token comes from this row
    if (bonus && !draws) return;                     // a bonus row that is not drawn from has nothing to do
    if (!draws && !P.grad) return;
    const RowConst rc = P.rowc[unit];
    const uint4* Trow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.T) + (size_t)unit * P.Vs);
    const uint4* Drow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.D) + (size_t)(b * P.k + (bonus ? 0 : i)) * P.Vs);
    ET* Grow = (P.grad && !bonus) ? reinterpret_cast<ET*>(P.grad) + (size_t)(b * P.k + i) * P.Vs : nullptr;
    const int NV = P.Vs / VEC;
    float* rsum = P.region_sums + (size_t)b * 2 * P.NR;
    const int r0 = sl * kVpSliceRegions, r1 = min(P.NR, r0 + kVpSliceRegions);
    for (int r = r0 + warp; r < r1; r += kVpWarps) {
        const int v0 = r * kRegionVecs;
        const int nv = min(kRegionVecs, NV - v0);
        if (!SD_IN((long long)(v0 + nv) * VEC - 1, P.Vs, 61) || !SD_IN(unit, P.B * K1, 62)) continue;
        uint4 rt[kRegionRows], rd[kRegionRows];
#pragma unroll
        for (int g = 0; g < kRegionRows; ++g) {
            const int vi = g * 32 + lane;
            rt[g] = vi < nv ? __ldcs(Trow + v0 + vi) : E::masked();
            rd[g] = (!bonus && vi < nv) ? __ldcs(Drow + v0 + vi) : E::masked();
        }
        const float mass = bonus ? pass2_region<DT, true>(rt, rd, nv, lane, P.c, rc, nullptr)
                                 : pass2_region<DT, false>(rt, rd, nv, lane, P.c, rc, Grow ? Grow + (size_t)v0 * VEC : nullptr);
        if (draws) {
            // mass of p_n in the region as well: a rejection whose residual has no mass draws from p_n
            float pm = 0.f;
            if (!bonus) {
#pragma unroll
                for (int g = 0; g < kRegionRows; ++g) {
                    float tv[VEC];
                    E::unpack(rt[g], tv);
                    if (g * 32 + lane < nv) {
#pragma unroll
                        for (int e = 0; e < VEC; ++e) pm += prob_elem(tv[e], P.c, rc);
                    }
                }
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) pm += __shfl_xor_sync(0xffffffffu, pm, off);
            }
            if (lane == 0) { rsum[r] = mass; rsum[P.NR + r] = pm; }
        }
    }
}

// This shard's share of the mass of the row the extra token is drawn from (fixed order, fp64).
__global__ void __launch_bounds__(32) sd_vp_mass_kernel(const VpParams P) {
    const int b = blockIdx.x, lane = threadIdx.x;
    const int per = (P.NR + 31) / 32;
    const int j0 = min(P.NR, lane * per), j1 = min(P.NR, j0 + per);
    for (int which = 0; which < 2; ++which) {
        const float* rs = P.region_sums + ((size_t)b * 2 + which) * P.NR;
        double mine = 0.0;
        for (int j = j0; j < j1; ++j) mine += (double)rs[j];
        const double incl = warp_inclusive_scan(mine);
        if (lane == 31) P.local_mass[b * 2 + which] = incl;
    }
}

// ---- phase 3 -------------------------------------------------------------------------------
// One warp per sequence.  Shares in rank order: the first rank whose running sum exceeds
// u_k * total owns the draw (the last rank with mass, if rounding leaves none).
template <int DT>
__global__ void __launch_bounds__(32) sd_vp_draw_kernel(const VpParams P) {
    constexpr int PER = kRegionVecs * Elem<DT>::VEC / 32;
    const int b = blockIdx.x, lane = threadIdx.x;
    const int k = P.k, K1 = k + 1;
    const int n = P.accept_len[b];
    const bool bonus = (n == k);
    uint32_t flags = 0;
    int which = 0;
    double total = 0.0;
    for (int g = 0; g < P.G; ++g) total += P.all_mass[((size_t)g * P.B + b) * 2];
    if (!bonus && !(total > 0.0)) {
        // a rejection whose residual has no mass on any rank (q = p and a forced rejection): the extra
        // token comes from p_n, and the status says so
        flags |= SD_STATUS_ZERO_RESIDUAL;
        which = 1;
        total = 0.0;
        for (int g = 0; g < P.G; ++g) total += P.all_mass[((size_t)g * P.B + b) * 2 + 1];
    }
    const int mode = bonus ? 1 : (which ? 2 : 0);
    const double t = (double)P.u[b * K1 + k] * total;
    int owner = -1, last_with_mass = -1;
    double before = 0.0, run = 0.0;
    for (int g = 0; g < P.G; ++g) {
        const double m = P.all_mass[((size_t)g * P.B + b) * 2 + which];
        if (m > 0.0) last_with_mass = g;
        if (owner < 0 && run + m > t) { owner = g; before = run; }
        run += m;
    }
    bool past_end = false;
    if (owner < 0) { owner = last_with_mass; past_end = true; }
    int y = -1;
    if (!(total > 0.0) || !isfinite(total)) {
        // no mass anywhere (a row without a usable denominator): the first entry of the vocabulary
        // stands in, and the status says so
        flags |= SD_STATUS_BAD_ROW;
        if (P.rank == 0) y = 0;
    } else if (owner == P.rank) {
        // the search of the single-GPU resolver, with the mass of the ranks before this one in front
        Params Q;
        memset(&Q, 0, sizeof Q);
        Q.T = P.T; Q.D = P.D; Q.V = P.Vs; Q.c = P.c;
        const int unit = b * K1 + n;
        const RowConst rc = P.rowc[unit];
        const size_t offT = (size_t)unit * P.Vs, offD = (size_t)(b * k + (bonus ? 0 : n)) * P.Vs;
        const float* rs = P.region_sums + ((size_t)b * 2 + which) * P.NR;
        const int per = (P.NR + 31) / 32;
        const int j0 = min(P.NR, lane * per), j1 = min(P.NR, j0 + per);
        double mine = 0.0;
        for (int j = j0; j < j1; ++j) mine += (double)rs[j];
        const double incl = warp_inclusive_scan(mine);
        int cand = 0x7fffffff;
        double cand_prefix = 0.0;
        if (!past_end) {
            double r2 = before + (incl - mine);
            for (int j = j0; j < j1; ++j) {
                const double next = r2 + (double)rs[j];
                if (next > t) { cand = j; cand_prefix = r2; break; }
                r2 = next;
            }
        }
        const unsigned has = __ballot_sync(0xffffffffu, cand != 0x7fffffff);
        int region = -1;
        double prefix = 0.0;
        bool last_only = past_end;
        if (has) {
            const int src = __ffs(has) - 1;
            region = __shfl_sync(0xffffffffu, cand, src);
            prefix = __shfl_sync(0xffffffffu, cand_prefix, src);
        } else {
            last_only = true;                     // rounding: the last region of this shard that holds mass
            int lastr = -1;
            for (int j = j0; j < j1; ++j)
                if (rs[j] > 0.f) lastr = j;
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) lastr = max(lastr, __shfl_xor_sync(0xffffffffu, lastr, off));
            region = lastr;
        }
        int local = -1;
        if (region >= 0) {
            double rtot;
            local = search_region<DT, PER, true>(Q, rc, mode, offT, offD, region, prefix, t, last_only, &rtot);
            if (local < 0) local = search_region<DT, PER, true>(Q, rc, mode, offT, offD, region, 0.0, 0.0, true, &rtot);
        }
        y = P.v_offset + (local < 0 ? 0 : local);
    }
    if (lane == 0 && flags && P.status) atomicOr(P.status + b, flags);
    for (int i = lane; i <= k; i += 32)
        P.tokens[b * K1 + i] = (i < n) ? P.x[b * k + i] : (i == n ? y : -1);
}

}  // namespace sdv
