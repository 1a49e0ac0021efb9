// The two kernels of the verify-and-feedback step.
//
//   sd_stream_kernel   fast path.  A persistent kernel of thread-block clusters.  A cluster takes a
//                      contiguous range of (sequence, row) units, one after the other; each block
//                      of the cluster owns a contiguous slice of the vocabulary, cut into stages
//                      of 2 KiB per row that its 16 consumer warps take in turn.
//                      A slice is streamed through a ring of small shared-memory stages twice:
//                      pass 1 (maxima, then softmax sums relative to integer references) reads it
//                      from HBM, pass 2 (gradient out, residual mass) reads it again a few
//                      microseconds later, when it is still in L2, so HBM sees each logit once.
//                      Inside a block the warps are specialised:
//                        consumers  each works through its own stages, which it fetches itself into
//                                   a private ring of three slots with bulk asynchronous copies
//                                   (cp.async.bulk + mbarrier), always three stages ahead, across
//                                   passes and units; warps meet only once per unit and pass;
//                        statistics adds up the consumers' sums, exchanges the block's partial
//                                   with the other blocks of the cluster through distributed
//                                   shared memory (remote stores + remote mbarrier arrivals, no
//                                   cluster-wide barrier) and publishes the row constants;
//                        resolver   reports rows (loss, rejection test), takes the sequence's tickets when
//                                   the block leaves a sequence and, if they were the last ones,
//                                   draws the extra token.
//                      Pass 2 of a unit is scheduled after pass 1 of the next unit (lag 1), which
//                      hides the exchange.
//   sd_generic_kernel  any V and any alignment.  One block per unit, sweeps over global memory
//                      with element loads.  Same arithmetic, same workspace, same resolver.
//
// A unit is row i of sequence b: i < k pairs target row i with draft row i (Algorithm 1's
// rejection test, the KL loss of Eq. "kl_divergence" and its gradient); i == k is the bonus row.
// Every wait is bounded; nobody waits for another cluster.
#pragma once

#include "sd_device.cuh"

namespace sdv {

// ---- geometry of the fast path -------------------------------------------------------------
// A row is cut into stages of 128 16-byte vectors (2 KiB); a stage is also a sampling region.
// Block r of a cluster of C owns the stages [r*S, (r+1)*S) of every row it works on, S =
// ceil(stages per row / C); stage s of the slice belongs to consumer warp s % 16, so sixteen
// consecutive stages are worked on at the same time.  Every consumer warp has a ring of its own.
constexpr int kConsumerWarps = 16;
constexpr int kStageGroups = 4;                               // groups of 32 vectors in a stage
constexpr int kStageVecs = 32 * kStageGroups;                 // vectors of one row in a stage
constexpr int kStageRowBytes = kStageVecs * 16;               // 2 KiB of one row
constexpr int kStageBytes = 2 * kStageRowBytes;               // target part + draft part
constexpr int kWarpSlots = 3;                                 // stages a consumer warp has in flight or in use
constexpr int kRingSlots = kConsumerWarps * kWarpSlots;       // 48 slots, 192 KiB
constexpr int kDoneDepth = 4;                                 // units the resolver may lag behind
constexpr int kStatsWarp = 0, kResolverWarp = 1, kFirstConsumerWarp = 2;
constexpr int kStreamThreads = (kFirstConsumerWarp + kConsumerWarps) * 32;
constexpr int kGenericWarps = 8;
constexpr int kGenericThreads = kGenericWarps * 32;

// ---- PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Arrival on the barrier at the same shared-memory offset in block `rank` of the cluster; orders
// this thread's earlier (remote) stores before it at cluster scope.
__device__ __forceinline__ void mbar_arrive_remote(uint64_t* bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %1;\n\t"
        "mbarrier.arrive.release.cluster.shared::cluster.b64 _, [ra];\n\t}" ::"r"(smem_u32(bar)),
        "r"(rank)
        : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cta.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait of one thread.  It gives up after kWaitLimit polls or kWaitCycles clock cycles,
// whichever comes first, or as soon as another thread of the block has given up (*abort != 0);
// the caller then leaves its loop and the kernel returns.  A failed poll is followed by a short
// sleep, so that waiting warps leave the issue slots and the shared-memory pipe to working ones.
template <bool CLUSTER, bool SLEEP = false>
__device__ __forceinline__ bool mbar_wait_thread(uint64_t* bar, uint32_t parity, volatile int* abort) {
    long long t0 = 0;
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        if (SLEEP) __nanosleep(64);   // warps with long waits leave the issue slots to the others
        if ((it & 63u) == 63u) {
            if (*abort) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kWaitCycles) break;
        }
    }
    *abort = 1;
    return false;
}
// The same for a whole warp (all 32 lanes call it): every lane observes the barrier itself (a
// warp whose lanes part ways at a wait is slow to get back together), and all lanes get the same
// answer.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, mbar_wait_thread<false>(bar, parity, abort) ? 1 : 0) != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, mbar_wait_thread<true, true>(bar, parity, abort) ? 1 : 0) != 0;
}
__device__ __forceinline__ bool mbar_wait_sleepy(uint64_t* bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, mbar_wait_thread<false, true>(bar, parity, abort) ? 1 : 0) != 0;
}
// 1-D bulk copy global -> shared of this block, completion counted on `bar`, with an L2 eviction
// policy.  Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                          uint64_t* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// L2 policies: keep (a line that will be read again shortly) and the default.
__device__ __forceinline__ uint64_t policy_keep() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_normal() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ void fence_barrier_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void store_streaming(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// ---- the two passes over one stage held in shared memory ------------------------------------
// A stage is 4 vectors per lane and row.  All of them are loaded before any arithmetic; vectors
// past the end of the row read as -inf, which adds nothing to any sum and is never stored.

// Pass 1: the stage's maxima; if they raise the warp's integer references (RT, RD), the running
// sums move to the new references (exact: powers of two); then the stage's sums.
template <int DT, bool BONUS>
__device__ __forceinline__ void pass1_stage(const uint4* st, int nv, int lane, float c, float& RT, float& RD,
                                            LaneSums& ls) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    uint4 rt[kStageGroups], rd[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        const int vi = g * 32 + lane;
        rt[g] = vi < nv ? st[vi] : E::masked();
        if (!BONUS) rd[g] = vi < nv ? st[kStageVecs + vi] : E::masked();
    }
    float mT[kStageGroups], mD[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        float v[VEC];
        E::unpack(rt[g], v);
        mT[g] = tree_max<VEC>(v);
        if (!BONUS) {
            E::unpack(rd[g], v);
            mD[g] = tree_max<VEC>(v);
        }
    }
    const float nT = fmaxf(RT, warp_max_ref(ref_of(fmaxf(fmax3(mT[0], mT[1], mT[2]), mT[3]), c)));
    const float nD = BONUS ? kEmptyRef : fmaxf(RD, warp_max_ref(ref_of(fmaxf(fmax3(mD[0], mD[1], mD[2]), mD[3]), c)));
    if (nT > RT || nD > RD) {
        ls.rescale(nT - RT, nD - RD);
        RT = nT;
        RD = nD;
    }
    float pT[kStageGroups], pD[kStageGroups], pW[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        float tv[VEC];
        E::unpack(rt[g], tv);
        if (!BONUS) {
            float dv[VEC];
            E::unpack(rd[g], dv);
            LaneSums::vector_pair<VEC>(tv, dv, c, -RT, -RD, pT[g], pD[g], pW[g]);
        } else {
            pT[g] = LaneSums::vector_bonus<VEC>(tv, c, -RT);
        }
    }
    ls.sT += (pT[0] + pT[1]) + (pT[2] + pT[3]);
    if (!BONUS) {
        ls.sD += (pD[0] + pD[1]) + (pD[2] + pD[3]);
        ls.w += (pW[0] + pW[1]) + (pW[2] + pW[3]);
    }
}

// Pass 2: gradient out (gdst = where the stage's part of the gradient row starts, or null) and
// the stage's mass (sum of max(0,p-q)/tau, or of p on the bonus row), in every lane.
template <int DT, bool BONUS>
__device__ __forceinline__ float pass2_stage(const uint4* st, int nv, int lane, float c, const RowConst& rc,
                                             typename Elem<DT>::type* gdst) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    uint4 rt[kStageGroups], rd[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        const int vi = g * 32 + lane;
        rt[g] = vi < nv ? st[vi] : E::masked();
        if (!BONUS) rd[g] = vi < nv ? st[kStageVecs + vi] : E::masked();
    }
    float ms[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        const int vi = g * 32 + lane;
        float tv[VEC], r[VEC];
        E::unpack(rt[g], tv);
        if (!BONUS) {
            float dv[VEC], gv[VEC];
            E::unpack(rd[g], dv);
#pragma unroll
            for (int z = 0; z < VEC; ++z) {
                gv[z] = grad_elem(tv[z], dv[z], c, rc);
                r[z] = fmaxf(-gv[z], 0.f);
            }
            if (gdst && vi < nv) store_streaming(gdst + (size_t)vi * VEC, E::pack(gv));
        } else {
#pragma unroll
            for (int z = 0; z < VEC; ++z) r[z] = prob_elem(tv[z], c, rc);
        }
        ms[g] = tree_sum<VEC>(r);
    }
    float mass = (ms[0] + ms[1]) + (ms[2] + ms[3]);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
    return mass;
}

// Control block of the fast path; lives in dynamic shared memory after the ring.
struct StreamShared {
    uint64_t full[kRingSlots];          // stage filled by the bulk copies        (1 arrival + bytes)
    uint64_t s1_done[2];                // consumers' sums of a unit posted       (consumer warps)
    uint64_t xchg_bar[2];               // partials of every block have arrived   (cluster size, remote)
    uint64_t rc_ready[2];               // row constants published                (1)
    uint64_t s2_done[kDoneDepth];       // unit finished in this block            (consumer warps + 1)
    uint64_t res_free[kDoneDepth];      // resolver is done with the unit         (1)
    float lane_sums[2][3][kConsumerWarps][33];        // sT, sD, w of every consumer lane (33: no bank conflicts)
    float warp_ref[2][kConsumerWarps][2];             // RT, RD each consumer warp used
    PartialStats wpart[kConsumerWarps]; // the consumer warps' partials of the unit being merged
    PartialStats xchg[2][kMaxCluster];  // written by every block of the cluster (distributed shared memory)
    PartialStats row[kDoneDepth];       // statistics of the whole row, for the row report
    RowConst rc[2];
    RowConst rc_done[kDoneDepth];       // the same, kept for the row report
    int abort;                          // a bounded wait gave up somewhere in this block
};

// Units [u0, u0+n) of cluster `cid` of `G`: contiguous, sizes differ by at most one.
__device__ __host__ __forceinline__ void cluster_units(int units, int G, int cid, int& u0, int& n) {
    const int base = units / G, rem = units % G;
    n = base + (cid < rem ? 1 : 0);
    u0 = cid * base + (cid < rem ? cid : rem);
}

// The passes of a block in the order in which it streams them: with lag 1,
// S1(0) S1(1) S2(0) S1(2) S2(1) ... S1(n-1) S2(n-2) S2(n-1); with lag 0, S1(0) S2(0) S1(1) ...
struct PassOrder {
    int nu, lag;
    __device__ __forceinline__ int count() const { return 2 * nu; }
    __device__ __forceinline__ int index_s1(int j) const { return lag ? (j == 0 ? 0 : 2 * j - 1) : 2 * j; }
    __device__ __forceinline__ int index_s2(int j) const { return lag ? (j == nu - 1 ? 2 * nu - 1 : 2 * j + 2) : 2 * j + 1; }
    // unit and kind (0 = pass 1, 1 = pass 2) of pass p
    __device__ __forceinline__ void decode(int p, int& j, int& kind) const {
        if (!lag) { j = p >> 1; kind = p & 1; return; }
        if (p == 0) { j = 0; kind = 0; }
        else if (p == 2 * nu - 1) { j = nu - 1; kind = 1; }
        else if (p & 1) { j = (p + 1) >> 1; kind = 0; }
        else { j = (p >> 1) - 1; kind = 1; }
    }
};

// ---- fast path -----------------------------------------------------------------------------
// lag: 1 if pass 2 of a unit is scheduled after pass 1 of the next unit, else 0.
template <int DT>
__global__ void __launch_bounds__(kStreamThreads, 1)
sd_stream_kernel(const __grid_constant__ Params P, const int lag) {
    using E = Elem<DT>;
    using ET = typename E::type;
    constexpr int VEC = E::VEC;
    constexpr int R = kRingSlots;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;
    StreamShared& sh = *reinterpret_cast<StreamShared*>(dyn_smem + (size_t)R * kStageBytes);

    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int G = (int)gridDim.x / C;             // clusters in the grid
    const int cid = (int)blockIdx.x / C;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int K1 = P.k + 1;
    int u0, nu;
    cluster_units(P.B * K1, G, cid, u0, nu);      // this cluster works on units u0 .. u0+nu-1

    const int NV = P.V / VEC;                     // vectors per row
    const int stages_row = (NV + kStageVecs - 1) / kStageVecs;   // = sampling regions per row
    const int stages_blk = (stages_row + C - 1) / C;
    const int s0 = rank * stages_blk;             // first stage (region) of this block's slice
    const int ns = max(0, min(stages_row - s0, stages_blk));     // stages of a pass
    const int vb0 = s0 * kStageVecs;              // first vector of the slice
    const int nvb = max(0, min(NV - vb0, ns * kStageVecs));
    const PassOrder order{nu, lag};
    volatile int* abort = &sh.abort;

    if (tid == 0) {
        for (int s = 0; s < R; ++s) mbar_init(&sh.full[s], 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sh.s1_done[s], kConsumerWarps);
            mbar_init(&sh.xchg_bar[s], (uint32_t)C);
            mbar_init(&sh.rc_ready[s], 1);
        }
        for (int s = 0; s < kDoneDepth; ++s) {
            mbar_init(&sh.s2_done[s], kConsumerWarps + 1);
            mbar_init(&sh.res_free[s], 1);
        }
        sh.abort = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    // every block of the cluster has initialised its barriers before anyone arrives on them
    cluster.sync();

    if (warp == kStatsWarp) {
        // ---- statistics: block partial -> cluster exchange -> row constants
        for (int j = 0; j < nu; ++j) {
            const int unit = u0 + j;
            const bool bonus = (unit % K1 == P.k);
            const int par = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const int dslot = j % kDoneDepth;
            if (!mbar_wait_sleepy(&sh.s1_done[par], ph, abort)) break;
            // lane l adds up half of the lanes of consumer warp l%16 (they share that warp's
            // references) in fp64; the 16 warp partials then meet in shared memory
            {
                const int w = lane & 15, h0 = (lane >> 4) * 16;
                double sT = 0.0, sD = 0.0, wv = 0.0;
#pragma unroll
                for (int l = 0; l < 16; ++l) {
                    sT += (double)sh.lane_sums[par][0][w][h0 + l];
                    sD += (double)sh.lane_sums[par][1][w][h0 + l];
                    wv += (double)sh.lane_sums[par][2][w][h0 + l];
                }
                sT += shfl_xor_f64(sT, 16);
                sD += shfl_xor_f64(sD, 16);
                wv += shfl_xor_f64(wv, 16);
                if (lane < kConsumerWarps) {
                    PartialStats wp;
                    wp.RT = sh.warp_ref[par][w][0];
                    wp.RD = sh.warp_ref[par][w][1];
                    wp.sT = sT; wp.sD = sD; wp.w = wv;
                    sh.wpart[lane] = wp;
                }
            }
            __syncwarp();
            const PartialStats mine = merge_partials_serial(sh.wpart, kConsumerWarps);
            __syncwarp();
            if (lane < C) {
                *cluster.map_shared_rank(&sh.xchg[par][rank], lane) = mine;
                mbar_arrive_remote(&sh.xchg_bar[par], (uint32_t)lane);
            }
            if (!mbar_wait_cluster(&sh.xchg_bar[par], ph, abort)) break;
            const PartialStats row = merge_partials_serial(sh.xchg[par], C);
            const RowConst rcw = row_constants(P, bonus, row);
            if (lane == 0) {
                sh.rc[par] = rcw;
                mbar_arrive(&sh.rc_ready[par]);
                // for the row report by the resolver: wait until it is done with the slot's last use
                bool ok = true;
                if (j >= kDoneDepth)
                    ok = mbar_wait_thread<false>(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, abort);
                if (ok) {
                    sh.row[dslot] = row;
                    sh.rc_done[dslot] = rcw;
                    mbar_arrive(&sh.s2_done[dslot]);
                }
            }
            if (__any_sync(0xffffffffu, *abort)) break;
        }
    } else if (warp == kResolverWarp) {
        // ---- resolver: row reports, tickets; the sequence's last tickets draw the token
        int seg = 0;                               // units of the current sequence finished so far
        for (int j = 0; j < nu; ++j) {
            const int unit = u0 + j;
            const int b = unit / K1, i = unit - b * K1;
            const bool bonus = (i == P.k);
            const int dslot = j % kDoneDepth;
            const bool reports = (j % C == rank);   // the blocks of the cluster take turns
            AcceptOperands aop;
            aop.valid = false;
            if (reports && lane == 0 && !bonus) aop = load_accept_operands<DT>(P, b, i);
            if (!mbar_wait_sleepy(&sh.s2_done[dslot], (uint32_t)(j / kDoneDepth) & 1u, abort)) break;
            if (reports && lane == 0) finish_row(P, b, i, sh.row[dslot], sh.rc_done[dslot], aop);
            __syncwarp();
            ++seg;
            const bool leaves = (i == P.k) || (j == nu - 1);   // last unit of the sequence in this cluster
            if (leaves) {
                int last = 0;
                if (lane == 0) last = take_tickets(P, b, (uint32_t)seg) ? 1 : 0;
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) resolve_sequence<DT>(P, b);
                seg = 0;
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
        }
    } else {
        // ---- consumers: warp cw owns stages cw, cw+16, ... of every pass; a stage is a sampling
        // region.  The warp walks its stages of all passes in order; stage number n of that walk
        // goes to slot n % 3 of the warp's own ring, and its copies are issued by the warp's first
        // lane as soon as stage n-3 has been worked on, whatever pass or unit it belongs to.
        const int cw = warp - kFirstConsumerWarp;
        const int nst = cw < ns ? (ns - cw + kConsumerWarps - 1) / kConsumerWarps : 0;   // my stages per pass
        const int n_total = order.count() * nst;
        unsigned char* myring = ring + (size_t)cw * kWarpSlots * kStageBytes;
        uint64_t* myfull = &sh.full[cw * kWarpSlots];
        const uint64_t keep = policy_keep(), normal = policy_normal();
        // issue cursor (lane 0 only): next stage to fetch, and where it lies
        int ni = 0, pi = 0, ti = 0;
        const ET* Tbase = nullptr;
        const ET* Dbase = nullptr;
        int kind_i = 0;
        auto issue_next = [&]() {     // lane 0
            if (ni >= n_total) return;
            if (ti == 0) {            // first stage of a pass: where the pass reads from
                int j;
                order.decode(pi, j, kind_i);
                const int unit = u0 + j;
                const int b = unit / K1, i = unit - b * K1;
                Tbase = reinterpret_cast<const ET*>(P.T) + (size_t)unit * P.V + (size_t)vb0 * VEC;
                Dbase = (i == P.k) ? nullptr
                                   : reinterpret_cast<const ET*>(P.D) + (size_t)(b * P.k + i) * P.V + (size_t)vb0 * VEC;
            }
            const int s = cw + ti * kConsumerWarps;
            const int v0 = s * kStageVecs;
            const uint32_t bytes = (uint32_t)min(kStageVecs, nvb - v0) * 16u;
            const int slot = ni % kWarpSlots;
            unsigned char* dst = myring + (size_t)slot * kStageBytes;
            const uint64_t pol = kind_i == 0 ? keep : normal;
            mbar_expect_tx(&myfull[slot], Dbase ? 2u * bytes : bytes);
            bulk_load(dst, Tbase + (size_t)v0 * VEC, bytes, &myfull[slot], pol);
            if (Dbase) bulk_load(dst + kStageRowBytes, Dbase + (size_t)v0 * VEC, bytes, &myfull[slot], pol);
            ++ni;
            if (++ti == nst) { ti = 0; ++pi; }
        };
        if (lane == 0)
            for (int t = 0; t < kWarpSlots; ++t) issue_next();
        int n = 0;                    // consume cursor: stages worked on so far
        // hand the slot of stage n back and fetch stage n+3 into it
        auto recycle = [&]() {
            __syncwarp();
            if (lane == 0) {
                fence_proxy_async();   // the warp's reads of the slot come before the copy that refills it
                issue_next();
            }
            ++n;
        };
        bool ok = true;
        for (int j = 0; j < nu + lag && ok; ++j) {
            if (j < nu) {
                // pass 1 of unit j, stage by stage: the stage's maxima first; if they raise the warp's
                // integer references, the running sums move to the new references (exact: powers of
                // two); then the stage's sums.
                const bool bonus = ((u0 + j) % K1 == P.k);
                float RT = kEmptyRef, RD = kEmptyRef;
                LaneSums ls;
                ls.init();
                for (int s = cw; s < ns; s += kConsumerWarps) {
                    const int slot = n % kWarpSlots;
                    if (!mbar_wait(&myfull[slot], (uint32_t)(n / kWarpSlots) & 1u, abort)) { ok = false; break; }
                    const uint4* sT = reinterpret_cast<const uint4*>(myring + (size_t)slot * kStageBytes);
                    const int nv = min(kStageVecs, nvb - s * kStageVecs);     // vectors of this stage
                    if (bonus) pass1_stage<DT, true>(sT, nv, lane, P.c, RT, RD, ls);
                    else       pass1_stage<DT, false>(sT, nv, lane, P.c, RT, RD, ls);
                    recycle();
                }
                if (!ok) break;
                const int parj = j & 1;
                sh.lane_sums[parj][0][cw][lane] = ls.sT;
                sh.lane_sums[parj][1][cw][lane] = ls.sD;
                sh.lane_sums[parj][2][cw][lane] = ls.w;
                if (lane == 0) { sh.warp_ref[parj][cw][0] = RT; sh.warp_ref[parj][cw][1] = RD; }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.s1_done[parj]);
            }
            if (j >= lag) {
                // pass 2 of unit j-lag: gradient out, mass of every stage (= sampling region)
                const int jj = j - lag;
                const int unit = u0 + jj;
                const int b = unit / K1, i = unit - b * K1;
                const bool bonus = (i == P.k);
                const int dslot = jj % kDoneDepth;
                if (!mbar_wait(&sh.rc_ready[jj & 1], (uint32_t)(jj >> 1) & 1u, abort)) { ok = false; break; }
                const RowConst rc = sh.rc[jj & 1];
                ET* Grow = (P.grad && !bonus)
                               ? reinterpret_cast<ET*>(P.grad) + (size_t)(b * P.k + i) * P.V + (size_t)vb0 * VEC
                               : nullptr;
                float* rsum = P.region_sums + (size_t)unit * P.NR + s0;
                for (int s = cw; s < ns; s += kConsumerWarps) {
                    const int slot = n % kWarpSlots;
                    if (!mbar_wait(&myfull[slot], (uint32_t)(n / kWarpSlots) & 1u, abort)) { ok = false; break; }
                    const uint4* sT = reinterpret_cast<const uint4*>(myring + (size_t)slot * kStageBytes);
                    const int nv = min(kStageVecs, nvb - s * kStageVecs);
                    const float mass = bonus ? pass2_stage<DT, true>(sT, nv, lane, P.c, rc, nullptr)
                                             : pass2_stage<DT, false>(sT, nv, lane, P.c, rc,
                                                                      Grow ? Grow + (size_t)s * kStageVecs * VEC : nullptr);
                    if (lane == 0) rsum[s] = mass;
                    recycle();
                }
                if (!ok) break;
                // the resolver's slot of unit jj-4 must be free again before this unit is reported done
                if (jj >= kDoneDepth &&
                    !mbar_wait(&sh.res_free[dslot], (uint32_t)(jj / kDoneDepth - 1) & 1u, abort)) { ok = false; break; }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
            }
        }
        // leaving early: no copy of this warp may still be in flight when the block returns
        if (!ok && lane == 0)
            for (int t = n; t < ni; ++t) {
                const uint32_t par = (uint32_t)(t / kWarpSlots) & 1u;
                for (uint32_t it = 0; it < kWaitLimit && !mbar_try_wait(&myfull[t % kWarpSlots], par); ++it) {}
            }
    }

    __syncthreads();
    if (sh.abort) {
        // a wait gave up: say so in every sequence this cluster has a unit of, and in every
        // sequence resolved from now on
        if (tid == 0) atomicExch(P.sticky, 1u);
        if (P.status)
            for (int j = tid; j < nu; j += kStreamThreads) atomicOr(P.status + (u0 + j) / K1, kStatusTimeout);
    }
    // no block leaves while another may still write to its shared memory
    cluster.sync();
}

// ---- generic path --------------------------------------------------------------------------
struct GenericShared {
    float wmax[2][kGenericWarps];
    PartialStats warp_part[kGenericWarps];
    RowConst rc;
    int last;
};

template <int DT>
__global__ void __launch_bounds__(kGenericThreads) sd_generic_kernel(const __grid_constant__ Params P) {
    using E = Elem<DT>;
    __shared__ GenericShared sh;

    const int unit = blockIdx.x;
    const int b = unit / (P.k + 1), i = unit % (P.k + 1);
    const bool bonus = (i == P.k);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t offT = (size_t)unit * P.V;
    const size_t offD = (size_t)(b * P.k + (bonus ? 0 : i)) * P.V;

    // sweep 0: the row maxima give the references of every exponential
    float mT = -3.402823466e+38f, mD = -3.402823466e+38f;
    for (int v = tid; v < P.V; v += kGenericThreads) {
        mT = fmaxf(mT, E::load(P.T, offT + v));
        if (!bonus) mD = fmaxf(mD, E::load(P.D, offD + v));
    }
    mT = warp_max_f32(mT);
    mD = warp_max_f32(mD);
    if (lane == 0) { sh.wmax[0][warp] = mT; sh.wmax[1][warp] = mD; }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < kGenericWarps; ++w) { mT = fmaxf(mT, sh.wmax[0][w]); mD = fmaxf(mD, sh.wmax[1][w]); }
    const float RT = ref_of(mT, P.c), RD = bonus ? kEmptyRef : ref_of(mD, P.c);

    // sweep 1: softmax sums
    LaneSums ls;
    ls.init();
    for (int v = tid; v < P.V; v += kGenericThreads) {
        float t[1] = {E::load(P.T, offT + v)};
        if (!bonus) {
            float d[1] = {E::load(P.D, offD + v)};
            ls.template add_pair<1>(t, d, P.c, -RT, -RD);
        } else {
            ls.template add_bonus<1>(t, P.c, -RT);
        }
    }
    {
        const PartialStats part = warp_sum_lanes(ls, RT, RD);
        if (lane == 0) sh.warp_part[warp] = part;
        __syncthreads();
        if (tid == 0) {
            const PartialStats row = merge_partials_serial(sh.warp_part, kGenericWarps);
            const RowConst rcw = row_constants(P, bonus, row);
            sh.rc = rcw;
            AcceptOperands aop;
            aop.valid = false;
            if (!bonus) aop = load_accept_operands<DT>(P, b, i);
            finish_row(P, b, i, row, rcw, aop);
        }
    }
    __syncthreads();
    const RowConst rc = sh.rc;

    // sweep 2: gradient and region sums, one sampling region per warp at a time
    float* rsum = P.region_sums + (size_t)unit * P.NR;
    for (int q = warp; q < P.NR; q += kGenericWarps) {
        const int ebase = q * P.RE;
        float mass = 0.f;
        for (int j = lane; j < P.RE; j += 32) {
            const int v = ebase + j;
            if (v < P.V) {
                const float t = E::load(P.T, offT + v);
                if (!bonus) {
                    const float d = E::load(P.D, offD + v);
                    const float g = grad_elem(t, d, P.c, rc);
                    mass += fmaxf(-g, 0.f);
                    if (P.grad) E::store(P.grad, offD + v, g);
                } else {
                    mass += prob_elem(t, P.c, rc);
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
        if (lane == 0) rsum[q] = mass;
    }

    // the block that takes the sequence's last ticket resolves it
    __syncthreads();
    if (tid == 0) sh.last = take_tickets(P, b, 1u) ? 1 : 0;
    __syncthreads();
    if (sh.last && warp == 0) resolve_sequence<DT>(P, b);
}

}  // namespace sdv
