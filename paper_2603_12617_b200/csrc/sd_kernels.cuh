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
// ceil(stages per row / C); stage s of the slice belongs to consumer warp s % 14, so fourteen
// consecutive stages are worked on at the same time.  Every consumer warp has a ring of its own.
constexpr int kConsumerWarps = 14;
constexpr int kStageGroups = 4;                               // groups of 32 vectors in a stage
constexpr int kStageVecs = 32 * kStageGroups;                 // vectors of one row in a stage
constexpr int kStageRowBytes = kStageVecs * 16;               // 2 KiB of one row
constexpr int kStageBytes = 2 * kStageRowBytes;               // target part + draft part
constexpr int kWarpSlots = 3;                                 // stages a consumer warp has in flight or in use
constexpr int kRingSlots = kConsumerWarps * kWarpSlots;       // 42 slots, 168 KiB
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
// 16 bytes to the same shared-memory offset in block `rank` of the cluster; their arrival is
// counted (as 16 bytes) on the barrier at offset `bar` of that block.  One-way: no acknowledgement.
__device__ __forceinline__ void st_async_remote(void* dst, uint64_t a, uint64_t b, uint64_t* bar, uint32_t rank) {
    asm volatile(
        "{\n\t.reg .b32 ra, rb;\n\t"
        "mapa.shared::cluster.u32 ra, %0, %4;\n\t"
        "mapa.shared::cluster.u32 rb, %1, %4;\n\t"
        "st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b64 [ra], {%2, %3}, [rb];\n\t}" ::"r"(
            smem_u32(dst)),
        "r"(smem_u32(bar)), "l"(a), "l"(b), "r"(rank)
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
// sleep (longer for the warps whose waits are long by design).
template <bool CLUSTER, int SLEEP_NS = 20>
__device__ __forceinline__ bool mbar_wait_thread(uint64_t* bar, uint32_t parity, volatile int* abort) {
    long long t0 = 0;
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
        __nanosleep(SLEEP_NS);   // waiting warps leave the issue slots to the working ones
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
    return __all_sync(0xffffffffu, mbar_wait_thread<true, 100>(bar, parity, abort) ? 1 : 0) != 0;
}
template <int SLEEP_NS>
__device__ __forceinline__ bool mbar_wait_sleepy(uint64_t* bar, uint32_t parity, volatile int* abort) {
    return __all_sync(0xffffffffu, mbar_wait_thread<false, SLEEP_NS>(bar, parity, abort) ? 1 : 0) != 0;
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
// A stage is kStageGroups vectors per lane and row.  All of them are loaded before any arithmetic; vectors
// past the end of the row read as -inf, which adds nothing to any sum and is never stored.

// Pass 1: the stage's softmax sums relative to the warp's integer references (RT, RD), added to
// the running sums.  References need not be the exact maxima: any integers work as long as nothing
// overflows, and sums under different references are merged exactly later.  So only the first
// stage of a unit looks for its maxima first; later stages reuse the references, and a stage whose
// sums come out too large for comfort (an entry far above everything the warp has seen: rare) is
// done again by pass1_stage_again after its maxima have raised the references and the running
// sums have moved with them (exact: powers of two).
struct Pass1State {
    float RT, RD;
    LaneSums ls;
};

// The stage's maxima raise the references; the running sums follow.
template <int DT, bool BONUS>
__device__ __forceinline__ void raise_references(const uint4 (&rt)[kStageGroups], const uint4 (&rd)[kStageGroups],
                                                 float c, Pass1State& s) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
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
    const float nT = fmaxf(s.RT, warp_max_ref(ref_of(tree_max<kStageGroups>(mT), c)));
    const float nD = BONUS ? kEmptyRef : fmaxf(s.RD, warp_max_ref(ref_of(tree_max<kStageGroups>(mD), c)));
    s.ls.rescale(nT - s.RT, nD - s.RD);
    s.RT = nT;
    s.RD = nD;
}

template <int DT, bool BONUS>
__device__ __forceinline__ void load_stage(const uint4* st, int nv, int lane, uint4 (&rt)[kStageGroups],
                                           uint4 (&rd)[kStageGroups]) {
    using E = Elem<DT>;
    if (nv == kStageVecs) {
#pragma unroll
        for (int g = 0; g < kStageGroups; ++g) {
            rt[g] = st[g * 32 + lane];
            if (!BONUS) rd[g] = st[kStageVecs + g * 32 + lane];
        }
    } else {
#pragma unroll
        for (int g = 0; g < kStageGroups; ++g) {
            const int vi = g * 32 + lane;
            rt[g] = vi < nv ? st[vi] : E::masked();
            if (!BONUS) rd[g] = vi < nv ? st[kStageVecs + vi] : E::masked();
        }
    }
}

// Returns only when every vector of the stage has arrived in this lane's registers (the value
// depends on all of them), so that the stage's slot may be overwritten afterwards.
template <bool BONUS>
__device__ __forceinline__ void await_stage_registers(const uint4 (&rt)[kStageGroups], const uint4 (&rd)[kStageGroups]) {
    uint32_t dep = 0;
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        dep ^= rt[g].w;
        if (!BONUS) dep ^= rd[g].w;
    }
    asm volatile("" ::"r"(dep) : "memory");
}

template <int DT, bool BONUS>
__device__ __forceinline__ void stage_sums(const uint4 (&rt)[kStageGroups], const uint4 (&rd)[kStageGroups], float c,
                                           float RT, float RD, float& sT, float& sD, float& sW) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    sT = sD = sW = 0.f;
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        float tv[VEC];
        E::unpack(rt[g], tv);
        if (!BONUS) {
            float dv[VEC], pT, pD, pW;
            E::unpack(rd[g], dv);
            LaneSums::vector_pair<VEC>(tv, dv, c, -RT, -RD, pT, pD, pW);
            sT += pT;
            sD += pD;
            sW += pW;
        } else {
            sT += LaneSums::vector_bonus<VEC>(tv, c, -RT);
        }
    }
}

// The slow way, out of line: maxima first, then the sums.  By now the stage's slot in the ring
// has been handed back, so the stage is read once more from global memory (gT, gD: where it
// starts in the two rows).
template <int DT, bool BONUS>
__device__ __noinline__ Pass1State pass1_stage_again(const uint4* gT, const uint4* gD, int nv, int lane, float c,
                                                     Pass1State s) {
    using E = Elem<DT>;
    uint4 rt[kStageGroups], rd[kStageGroups];
#pragma unroll
    for (int g = 0; g < kStageGroups; ++g) {
        const int vi = g * 32 + lane;
        rt[g] = vi < nv ? __ldg(gT + vi) : E::masked();
        if (!BONUS) rd[g] = vi < nv ? __ldg(gD + vi) : E::masked();
    }
    raise_references<DT, BONUS>(rt, rd, c, s);
    float sT, sD, sW;
    stage_sums<DT, BONUS>(rt, rd, c, s.RT, s.RD, sT, sD, sW);
    s.ls.sT += sT;
    s.ls.sD += sD;
    s.ls.w += sW;
    return s;
}

// `handed_back` is called once the stage is in registers: the caller refills the slot then.
template <int DT, bool BONUS, class F>
__device__ __forceinline__ void pass1_stage(const uint4* st, const uint4* gT, const uint4* gD, int nv, int lane, float c,
                                            bool first, Pass1State& s, F&& handed_back) {
    constexpr float kTooLarge = 1.152921504606846976e18f;   // 2^60
    uint4 rt[kStageGroups], rd[kStageGroups];
    load_stage<DT, BONUS>(st, nv, lane, rt, rd);
    await_stage_registers<BONUS>(rt, rd);
    handed_back();
    if (first) raise_references<DT, BONUS>(rt, rd, c, s);
    float sT, sD, sW;
    stage_sums<DT, BONUS>(rt, rd, c, s.RT, s.RD, sT, sD, sW);
    // (written so that a NaN counts as too large)
    if (!first && __any_sync(0xffffffffu, !(sT < kTooLarge) || !(sD < kTooLarge))) {
        s = pass1_stage_again<DT, BONUS>(gT, gD, nv, lane, c, s);
        return;
    }
    s.ls.sT += sT;
    s.ls.sD += sD;
    s.ls.w += sW;
}

// Pass 2: gradient out (gdst = where the stage's part of the gradient row starts, or null) and
// the stage's mass (sum of max(0,p-q)/tau, or of p on the bonus row), in every lane.
template <int DT, bool BONUS, class F>
__device__ __forceinline__ float pass2_stage(const uint4* st, int nv, int lane, float c, const RowConst& rc,
                                             typename Elem<DT>::type* gdst, F&& handed_back) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    uint4 rt[kStageGroups], rd[kStageGroups];
    load_stage<DT, BONUS>(st, nv, lane, rt, rd);
    await_stage_registers<BONUS>(rt, rd);
    handed_back();
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
            for (int z = 0; z < VEC; z += 2) {
                const float2 g2 = grad_elem2(make_float2(tv[z], tv[z + 1]), make_float2(dv[z], dv[z + 1]), c, rc);
                gv[z] = g2.x;
                gv[z + 1] = g2.y;
                r[z] = fmaxf(-g2.x, 0.f);
                r[z + 1] = fmaxf(-g2.y, 0.f);
            }
            if (gdst && vi < nv) store_streaming(gdst + (size_t)vi * VEC, E::pack(gv));
        } else {
#pragma unroll
            for (int z = 0; z < VEC; ++z) r[z] = prob_elem(tv[z], c, rc);
        }
        ms[g] = tree_sum<VEC>(r);
    }
    float mass = tree_sum<kStageGroups>(ms);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
    return mass;
}

// Control block of the fast path; lives in dynamic shared memory after the ring.
struct StreamShared {
    uint64_t full[kRingSlots];          // stage filled by the bulk copies        (1 arrival + bytes)
    uint64_t s1_done[2];                // consumers' sums of a unit posted       (consumer warps)
    uint64_t xchg_bar[2];               // partials of every block have arrived   (1 arrival + bytes, remote)
    uint64_t rc_ready[2];               // row constants published                (1)
    uint64_t s2_done[kDoneDepth];       // unit finished in this block            (consumer warps + 1)
    uint64_t res_free[kDoneDepth];      // resolver is done with the unit         (1)
    PartialStats wpart[2][kConsumerWarps];   // the consumer warps' partials of a unit
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

// The order in which a consumer warp walks its stages.  The warp has nst stages in every pass.
// Pass 2 of a unit needs the row constants, which take an exchange between the blocks of the
// cluster; so it is scheduled after the first L stages of pass 1 of the next unit:
//   S1(0)[0,nst)  then for j = 1 .. nu-1:  S1(j)[0,L)  S2(j-1)[0,nst)  S1(j)[L,nst)   then  S2(nu-1)[0,nst)
// The smaller L, the less data lies between the two passes (it has to stay in L2 meanwhile).

// ---- fast path -----------------------------------------------------------------------------
// lag_stages: stages (per consumer warp) of pass 1 of the next unit that go before pass 2 of a unit.
// ENS: the units are those of the ensemble feedback (see UnitRef); nothing is verified or drawn.
// STATS: pass 1 only -- row constants, losses and rejection tests of every row; no gradient, no
// masses, no draw (the error-position feedback finishes the one row it needs in a kernel of its own).
template <int DT, bool ENS, bool STATS = false>
__global__ void __launch_bounds__(kStreamThreads, 1)
sd_stream_kernel(const __grid_constant__ Params P, const int lag_stages) {
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
    // The plain step gives a cluster a contiguous range of units (the rows of a sequence stay
    // together: fewer tickets).  The ensemble deals its units round the clusters instead: the units
    // that read the same target row then run on neighbouring clusters at about the same time, and all
    // but the first find the row in L2.
    int u0, nu, ustep = 1;
    if constexpr (ENS) {
        const int units = total_units<true>(P);
        u0 = cid;
        ustep = G;
        nu = cid < units ? (units - cid + G - 1) / G : 0;
    } else {
        cluster_units(total_units<false>(P), G, cid, u0, nu);   // this cluster works on units u0 .. u0+nu-1
    }

    const int NV = P.V / VEC;                     // vectors per row
    const int stages_row = (NV + kStageVecs - 1) / kStageVecs;   // = sampling regions per row
    const int stages_blk = (stages_row + C - 1) / C;
    const int s0 = rank * stages_blk;             // first stage (region) of this block's slice
    const int ns = max(0, min(stages_row - s0, stages_blk));     // stages of a pass
    const int vb0 = s0 * kStageVecs;              // first vector of the slice
    const int nvb = max(0, min(NV - vb0, ns * kStageVecs));
    volatile int* abort = &sh.abort;

    if (tid == 0) {
        for (int s = 0; s < R; ++s) mbar_init(&sh.full[s], 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sh.s1_done[s], kConsumerWarps);
            mbar_init(&sh.xchg_bar[s], 1);
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
            const int unit = u0 + j * ustep;
            const bool bonus = !ENS && (unit % K1 == P.k);
            const int par = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const int dslot = j % kDoneDepth;
            if (lane == 0) mbar_expect_tx(&sh.xchg_bar[par], (uint32_t)C * (uint32_t)sizeof(PartialStats));
            if (!mbar_wait_sleepy<100>(&sh.s1_done[par], ph, abort)) break;
            // the block's partial from its 16 warp partials, then one copy to every block of the cluster
            const PartialStats mine = warp_merge_lanes(lane < kConsumerWarps ? sh.wpart[par][lane] : empty_partial());
            if (lane < C) {
                uint64_t refs;
                memcpy(&refs, &mine.RT, 8);
                PartialStats* dst = &sh.xchg[par][rank];
                st_async_remote(dst, refs, (uint64_t)__double_as_longlong(mine.sT), &sh.xchg_bar[par], (uint32_t)lane);
                st_async_remote(&dst->sD, (uint64_t)__double_as_longlong(mine.sD), (uint64_t)__double_as_longlong(mine.w),
                                &sh.xchg_bar[par], (uint32_t)lane);
            }
            if (!mbar_wait_cluster(&sh.xchg_bar[par], ph, abort)) break;
            const PartialStats row = warp_merge_lanes(lane < C ? sh.xchg[par][lane] : empty_partial());
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
            const int unit = u0 + j * ustep;
            const int dslot = j % kDoneDepth;
            const bool reports = (j % C == rank);   // the blocks of the cluster take turns
            if constexpr (ENS) {
                if (!mbar_wait_sleepy<500>(&sh.s2_done[dslot], (uint32_t)(j / kDoneDepth) & 1u, abort)) break;
                if (reports && lane == 0) finish_row_ensemble(P, unit_ref<true>(P, unit), sh.row[dslot]);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
                continue;
            }
            const int b = unit / K1, i = unit - b * K1;
            const bool bonus = (i == P.k);
            AcceptOperands aop;
            aop.valid = false;
            if (reports && lane == 0 && !bonus) aop = load_accept_operands<DT>(P, b, i);
            if (!mbar_wait_sleepy<500>(&sh.s2_done[dslot], (uint32_t)(j / kDoneDepth) & 1u, abort)) break;
            if (reports && lane == 0) finish_row(P, b, i, sh.row[dslot], sh.rc_done[dslot], aop);
            __syncwarp();
            if constexpr (STATS) {
                if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
                continue;
            }
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
        // region.  The warp walks its stages of all passes in a fixed order (Walk); stage number n
        // of that walk goes to slot n % 3 of the warp's own ring, and its copies are issued by the
        // warp's first lane as soon as stage n-3 has been worked on, whatever pass or unit it is of.
        const int cw = warp - kFirstConsumerWarp;
        const int nst = cw < ns ? (ns - cw + kConsumerWarps - 1) / kConsumerWarps : 0;   // my stages per pass
        if (nst == 0) {
            // no data of its own (short rows): the warp only keeps the per-unit protocol going
            for (int j = 0; j < nu; ++j) {
                if (lane == 0) { sh.wpart[j & 1][cw] = empty_partial(); mbar_arrive(&sh.s1_done[j & 1]); }
                const int dslot = j % kDoneDepth;
                if (!mbar_wait(&sh.rc_ready[j & 1], (uint32_t)(j >> 1) & 1u, abort)) break;
                if (j >= kDoneDepth && !mbar_wait(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, abort)) break;
                if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
            }
        } else {
            const int L = min(max(lag_stages, 0), nst);
            const int n_total = (STATS ? 1 : 2) * nu * nst;
            unsigned char* myring = ring + (size_t)cw * kWarpSlots * kStageBytes;
            uint64_t* myfull = &sh.full[cw * kWarpSlots];
            const uint64_t keep = policy_keep(), normal = policy_normal();
            // issue cursor (lane 0): the walk S1(0) | S1(j)[0,L) S2(j-1) S1(j)[L,nst) ... | S2(nu-1)
            // runs of the walk: 0 = S1(0), 1 = head of S1(ji), 2 = S2(ji-1), 3 = rest of S1(ji), 4 = S2(nu-1)
            int ni = 0, run = 0, ji = 0, ti = 0, endi = nst;   // stage number, run, unit of the run's pass 1, stage, end
            const ET* Tb = nullptr;       // where the next copy of the run reads from; Db null on a bonus row
            const ET* Db = nullptr;
            uint64_t pol = keep;
            int slot_i = 0;               // ring slot of the next copy
            constexpr size_t kStride = (size_t)kConsumerWarps * kStageVecs * VEC;   // from one of my stages to the next
            auto begin_run = [&]() {      // lane 0
                const UnitRef ur = unit_ref<ENS>(P, u0 + (run == 2 ? ji - 1 : run == 4 ? nu - 1 : ji) * ustep);
                const size_t off = (size_t)(vb0 + cw * kStageVecs) * VEC + (size_t)ti * kStride;
                Tb = reinterpret_cast<const ET*>(P.T) + ur.t_row * P.V + off;
                Db = ur.bonus ? nullptr : reinterpret_cast<const ET*>(ENS ? P.Dn[ur.n] : P.D) + ur.d_row * P.V + off;
                pol = (run == 2 || run == 4) ? normal : keep;
            };
            auto issue_next = [&]() {     // lane 0
                if (ni >= n_total) return;
                const uint32_t bytes = (uint32_t)min(kStageVecs, nvb - (cw + ti * kConsumerWarps) * kStageVecs) * 16u;
                unsigned char* dst = myring + (size_t)slot_i * kStageBytes;
                mbar_expect_tx(&myfull[slot_i], Db ? 2u * bytes : bytes);
                bulk_load(dst, Tb, bytes, &myfull[slot_i], pol);
                if (Db) { bulk_load(dst + kStageRowBytes, Db, bytes, &myfull[slot_i], pol); Db += kStride; }
                Tb += kStride;
                if (++slot_i == kWarpSlots) slot_i = 0;
                ++ni;
                ++ti;
                if (ti >= endi) {
                    while (ti >= endi && run != 5) {
                        // the next run that is not empty
                        constexpr int kLast = STATS ? 5 : 4;          // no pass 2 to fetch for in a pass-1-only walk
                        if (run == 0) { if (nu > 1) { run = 1; ji = 1; } else run = kLast; }
                        else if (run == 1) run = STATS ? 3 : 2;
                        else if (run == 2) run = 3;
                        else if (run == 3) { if (ji + 1 < nu) { run = 1; ++ji; } else run = kLast; }
                        else run = 5;
                        if (run == 1) { ti = 0; endi = L; }
                        else if (run == 3) { ti = L; endi = nst; }
                        else { ti = 0; endi = nst; }
                    }
                    if (run != 5) begin_run();
                }
            };
            if (lane == 0) begin_run();
            if (lane == 0)
                for (int t = 0; t < kWarpSlots; ++t) issue_next();
            int n = 0;                    // consume cursor: stages worked on so far, its slot and parity
            int slot_c = 0;
            uint32_t par_c = 0;
            bool ok = true;
            // The stage is in registers: hand its slot back and fetch stage n+3 of the walk into it.
            // (Every lane's loads from the slot have returned their values before the copy is issued.)
            auto recycle = [&]() {
                __syncwarp();
                if (lane == 0) issue_next();
                ++n;
                if (++slot_c == kWarpSlots) { slot_c = 0; par_c ^= 1u; }
            };
            Pass1State ps;
            ps.RT = ps.RD = kEmptyRef;
            ps.ls.init();
            auto run_pass1 = [&](int j, int t0, int t1) {
                const UnitRef ur = unit_ref<ENS>(P, u0 + j * ustep);
                const bool bonus = ur.bonus;
                // the block's slice of the two rows in global memory (for the rare second try of a stage)
                const ET* Trow = reinterpret_cast<const ET*>(P.T) + ur.t_row * P.V + (size_t)vb0 * VEC;
                const ET* Drow = reinterpret_cast<const ET*>(ENS ? P.Dn[ur.n] : P.D) + ur.d_row * P.V + (size_t)vb0 * VEC;
                for (int t = t0; t < t1 && ok; ++t) {
                    const int slot = slot_c;
                    if (!mbar_wait(&myfull[slot], par_c, abort)) { ok = false; break; }
                    const uint4* st = reinterpret_cast<const uint4*>(myring + (size_t)slot * kStageBytes);
                    const int s = cw + t * kConsumerWarps;
                    const int nv = min(kStageVecs, nvb - s * kStageVecs);     // vectors of this stage
                    const uint4* gT = reinterpret_cast<const uint4*>(Trow) + (size_t)s * kStageVecs;
                    const uint4* gD = reinterpret_cast<const uint4*>(Drow) + (size_t)s * kStageVecs;
                    if (bonus) pass1_stage<DT, true>(st, gT, gD, nv, lane, P.c, t == 0, ps, recycle);
                    else       pass1_stage<DT, false>(st, gT, gD, nv, lane, P.c, t == 0, ps, recycle);
                }
            };
            auto run_pass2 = [&](int j) {
                const int unit = u0 + j * ustep;
                const UnitRef ur = unit_ref<ENS>(P, unit);
                const bool bonus = ur.bonus;
                const int dslot = j % kDoneDepth;
                if (!mbar_wait(&sh.rc_ready[j & 1], (uint32_t)(j >> 1) & 1u, abort)) { ok = false; return; }
                const RowConst rc = sh.rc[j & 1];
                void* const gbase = ENS ? P.Gn[ur.n] : P.grad;
                ET* Grow = (gbase && !bonus) ? reinterpret_cast<ET*>(gbase) + ur.d_row * P.V + (size_t)vb0 * VEC : nullptr;
                float* rsum = ENS ? nullptr : P.region_sums + (size_t)unit * P.NR + s0;
                for (int t = 0; t < nst; ++t) {
                    const int slot = slot_c;
                    if (!mbar_wait(&myfull[slot], par_c, abort)) { ok = false; return; }
                    const uint4* st = reinterpret_cast<const uint4*>(myring + (size_t)slot * kStageBytes);
                    const int s = cw + t * kConsumerWarps;
                    const int nv = min(kStageVecs, nvb - s * kStageVecs);
                    const float mass = bonus ? pass2_stage<DT, true>(st, nv, lane, P.c, rc, nullptr, recycle)
                                             : pass2_stage<DT, false>(st, nv, lane, P.c, rc,
                                                                      Grow ? Grow + (size_t)s * kStageVecs * VEC : nullptr,
                                                                      recycle);
                    if (!ENS && lane == 0) rsum[s] = mass;
                }
                // the resolver's slot of unit j-4 must be free again before this unit is reported done
                if (j >= kDoneDepth &&
                    !mbar_wait(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, abort)) { ok = false; return; }
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
            };
            // The walk, segment by segment (each pass has one call site, which keeps the hot code small):
            // unit j contributes  [pass 1 head]  [pass 2 of unit j-1]  [pass 1 rest];  then pass 2 of the last unit.
            for (int seg = 0; seg <= 3 * nu && ok; ++seg) {
                const int j = seg / 3, kind = seg - 3 * j;
                int p1 = -1, p2 = -1, t0 = 0, t1 = 0;
                const int head = (j == 0) ? nst : L;
                if (j == nu) p2 = nu - 1;
                else if (kind == 0) { p1 = j; t0 = 0; t1 = head; }
                else if (kind == 1) { if (j > 0) p2 = j - 1; }
                else { p1 = j; t0 = head; t1 = nst; }
                if (p2 >= 0) {
                    if constexpr (STATS) {
                        // nothing to do for the unit but to report it finished -- after its row
                        // constants are out, as in the full walk: the statistics warp is then done
                        // with the partials of the unit, whose slots the unit after next reuses
                        const int dslot = p2 % kDoneDepth;
                        if (!mbar_wait(&sh.rc_ready[p2 & 1], (uint32_t)(p2 >> 1) & 1u, abort)) { ok = false; break; }
                        if (p2 >= kDoneDepth &&
                            !mbar_wait(&sh.res_free[dslot], (uint32_t)(p2 / kDoneDepth - 1) & 1u, abort)) { ok = false; break; }
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
                    } else {
                        run_pass2(p2);
                    }
                }
                if (p1 >= 0) {
                    run_pass1(p1, t0, t1);
                    if (ok && kind == 2) {
                        // pass 1 of the unit is over: the warp's partial for the statistics warp
                        const PartialStats part = warp_sum_lanes(ps.ls, ps.RT, ps.RD);
                        if (lane == 0) {
                            sh.wpart[j & 1][cw] = part;
                            mbar_arrive(&sh.s1_done[j & 1]);
                        }
                        ps.RT = ps.RD = kEmptyRef;
                        ps.ls.init();
                    }
                }
            }
            // leaving early: no copy of this warp may still be in flight when the block returns
            if (!ok && lane == 0)
                for (int t = n; t < ni; ++t) {
                    const uint32_t par = (uint32_t)(t / kWarpSlots) & 1u;
                    for (uint32_t it = 0; it < kWaitLimit && !mbar_try_wait(&myfull[t % kWarpSlots], par); ++it) {}
                }
        }
    }

    __syncthreads();
    if (sh.abort) {
        // a wait gave up: say so in every sequence this cluster has a unit of, and in every
        // sequence resolved from now on
        if (tid == 0) atomicExch(P.sticky, 1u);
        if (P.status)
            for (int j = tid; j < nu; j += kStreamThreads) atomicOr(P.status + unit_ref<ENS>(P, u0 + j * ustep).b, kStatusTimeout);
    }
    // no block leaves while another may still write to its shared memory
    cluster.sync();
}

// ---- generic path --------------------------------------------------------------------------
struct GenericShared {
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

    // sweep 1: softmax sums relative to integer references that every warp raises as it goes (the
    // sums follow by exact powers of two), eight entries per thread at a time; the warps' partial
    // sums, each under its own references, are merged exactly afterwards
    constexpr int kPer = (DT == SD_DTYPE_BF16) ? 16 : 8;
    float RT = kEmptyRef, RD = kEmptyRef;
    LaneSums ls;
    ls.init();
    for (int base = 0; base < P.V; base += kPer * kGenericThreads) {
        float t[kPer], d[kPer];
#pragma unroll
        for (int j = 0; j < kPer; ++j) {
            const int v = base + j * kGenericThreads + tid;
            t[j] = v < P.V ? E::load(P.T, offT + v) : -INFINITY;
            d[j] = (!bonus && v < P.V) ? E::load(P.D, offD + v) : -INFINITY;
        }
        float mt = t[0], md = d[0];
#pragma unroll
        for (int j = 1; j < kPer; ++j) { mt = fmaxf(mt, t[j]); md = fmaxf(md, d[j]); }
        const float nT = fmaxf(RT, warp_max_ref(ref_of(mt, P.c)));
        const float nD = bonus ? kEmptyRef : fmaxf(RD, warp_max_ref(ref_of(md, P.c)));
        ls.rescale(nT - RT, nD - RD);
        RT = nT;
        RD = nD;
#pragma unroll
        for (int j0 = 0; j0 < kPer; j0 += 8) {
            float t8[8], d8[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) { t8[j] = t[j0 + j]; d8[j] = d[j0 + j]; }
            if (!bonus) ls.template add_pair<8>(t8, d8, P.c, -RT, -RD);
            else        ls.template add_bonus<8>(t8, P.c, -RT);
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
#pragma unroll 8
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

// ---- online ensemble ---------------------------------------------------------------------
// Mean loss of the round per learner (fixed summation order), cumulative losses, Hedge weights.
__global__ void __launch_bounds__(256) sd_hedge_kernel(const float* loss, int N, long long per, double eps,
                                                       const double* cum_in, double* round_loss, double* cum_out,
                                                       float* weights, const uint32_t* sticky, uint32_t* status,
                                                       int B) {
    __shared__ double part[256];
    __shared__ double mean[kMaxLearners];
    const int tid = threadIdx.x;
    for (int n = 0; n < N; ++n) {
        double s = 0.0;
        for (long long j = tid; j < per; j += 256) s += (double)loss[(size_t)n * per + j];
        part[tid] = s;
        __syncthreads();
        for (int w = 128; w > 0; w >>= 1) {
            if (tid < w) part[tid] += part[tid + w];
            __syncthreads();
        }
        if (tid == 0) mean[n] = part[0] / (double)per;
        __syncthreads();
    }
    if (tid == 0) {
        double cum[kMaxLearners], lowest = INFINITY, Z = 0.0;
        for (int n = 0; n < N; ++n) {
            cum[n] = (cum_in ? cum_in[n] : 0.0) + mean[n];
            if (cum[n] < lowest) lowest = cum[n];
        }
        for (int n = 0; n < N; ++n) Z += exp(-eps * (cum[n] - lowest));
        for (int n = 0; n < N; ++n) {
            round_loss[n] = mean[n];
            cum_out[n] = cum[n];
            weights[n] = (float)(exp(-eps * (cum[n] - lowest)) / Z);
        }
    }
    // a bounded wait gave up somewhere in the feedback kernel: nothing of this round is valid
    if (status && *sticky != 0)
        for (int b = tid; b < B; b += 256) atomicOr(status + b, kStatusTimeout);
}

}  // namespace sdv
