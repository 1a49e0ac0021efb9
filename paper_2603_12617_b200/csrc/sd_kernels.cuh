// The two kernels of the verify-and-feedback step.
//
//   sd_stream_kernel   fast path.  A persistent kernel of thread-block clusters, one block of 32
//                      warps per SM.  A cluster takes a contiguous range of (sequence, row) units,
//                      one after the other; each block of the cluster owns a contiguous slice of
//                      the vocabulary, cut into sampling regions of 64 16-byte vectors (1 KiB of a
//                      row) and into stages of 28 regions (28 KiB of the target row and 28 KiB of
//                      the draft row).  A slice goes through a ring of shared-memory stages twice:
//                      pass 1 (softmax sums relative to integer references) brings it from HBM and
//                      asks L2 to hold on to it, pass 2 (gradient out, residual mass) fetches it
//                      again a few microseconds later, last stage first, when it is still in L2,
//                      so HBM sees each logit once.  Inside a block the warps are specialised:
//                        producer   two threads fetch the stages of the walk, in order, with bulk
//                                   asynchronous copies (cp.async.bulk + mbarrier): the first arms
//                                   the stage's barrier and copies the target part, the second
//                                   copies the draft part, each as soon as the consumers have
//                                   handed the slot back;
//                        consumers  28 warps; warp w takes region w of every stage into registers,
//                                   hands its share of the slot back at once and works from
//                                   registers; warps meet only through the ring's barriers and
//                                   once per unit and pass;
//                        statistics adds up the consumers' sums, exchanges the block's partial
//                                   with the other blocks of the cluster through distributed
//                                   shared memory (remote stores + remote mbarrier arrivals, no
//                                   cluster-wide barrier) and publishes the row constants;
//                        resolver   reports rows (loss, rejection test), takes the sequence's tickets when
//                                   the block leaves a sequence and, if they were the last ones,
//                                   draws the extra token.
//                      Pass 2 of a unit is scheduled after the first stages of pass 1 of the next
//                      unit (the lag), which hides the exchange.
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
// A row is cut into sampling regions of kRegionVecs 16-byte vectors; block r of a cluster of C owns
// the regions [r*S, (r+1)*S) of every row it works on, S = ceil(regions per row / C).  A stage is
// kConsumerWarps consecutive regions of the slice, one per consumer warp: 28 KiB of the target row
// and 28 KiB of the draft row, fetched by one bulk copy each.
constexpr int kHelperWarps = 4;                               // statistics, resolver, producer, one idle
constexpr int kConsumerWarps = 28;
constexpr int kStageVecs = kConsumerWarps * kRegionVecs;      // vectors of one row in a stage
constexpr int kStageRowBytes = kStageVecs * 16;               // 28 KiB of one row
constexpr int kStageBytes = 2 * kStageRowBytes;               // target part + draft part
constexpr int kRingStages = 4;                                // most stages a ring has (224 KiB)
// Stages of the ring by element type: measured, the fourth stage gains 4 % on the largest fp32 workload
// and loses 3 % on the bf16 ones.
template <int DT> struct RingStages { static constexpr int value = DT == SD_DTYPE_F32 ? 4 : 3; };
constexpr int kDoneDepth = 3;                                 // units the resolver may lag behind
constexpr int kStatsWarp = 0, kResolverWarp = 1, kProducerWarp = 2, kFirstConsumerWarp = kHelperWarps;
constexpr int kStreamThreads = (kHelperWarps + kConsumerWarps) * 32;
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
// Counts `bytes` as transferred on the barrier without a copy (the checked build's stand-in for a
// copy that it refused to issue).
__device__ __forceinline__ void mbar_complete_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.complete_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
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
// Non-blocking: has the phase of that parity completed?  (try_wait may suspend the thread for a while.)
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.acquire.cta.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
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
// Bounded wait of one thread.  It gives up after `limit` polls or kWaitCycles clock cycles,
// whichever comes first, or as soon as another thread of the block has given up (*abort != 0);
// the caller then leaves its loop and the kernel returns.  A failed poll is followed by a short
// sleep (longer for the warps whose waits are long by design).
struct WaitCtx {
    volatile int* abort;
    uint32_t limit;
};
template <bool CLUSTER, int SLEEP_NS = 20>
__device__ __forceinline__ bool mbar_wait_thread(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    volatile int* abort = wc.abort;
    long long t0 = 0;
    // (A limit of a few polls is a caller asking for waits that give up at once: those polls only
    // look, where the usual ones let the hardware suspend the thread until the phase ends or a
    // time limit of its own runs out.)
    const bool look_only = wc.limit < 64u;
    for (uint32_t it = 0; it < wc.limit; ++it) {
        if (look_only ? mbar_test(bar, parity)
                      : (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity))) return true;
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
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    return __all_sync(0xffffffffu, mbar_wait_thread<false>(bar, parity, wc) ? 1 : 0) != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    return __all_sync(0xffffffffu, mbar_wait_thread<true, 100>(bar, parity, wc) ? 1 : 0) != 0;
}
template <int SLEEP_NS>
__device__ __forceinline__ bool mbar_wait_sleepy(uint64_t* bar, uint32_t parity, const WaitCtx& wc) {
    return __all_sync(0xffffffffu, mbar_wait_thread<false, SLEEP_NS>(bar, parity, wc) ? 1 : 0) != 0;
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
// Bulk prefetch global -> L2 (no shared-memory destination, nothing to wait for).  Address 16-byte
// aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_prefetch_l2(const void* src_gmem, uint32_t bytes, uint64_t policy) {
    asm volatile("cp.async.bulk.prefetch.L2.global.L2::cache_hint [%0], %1, %2;" ::"l"(src_gmem), "r"(bytes), "l"(policy)
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

// L2 policy for data nobody will read again (the second pass): first in line for eviction.
__device__ __forceinline__ uint64_t policy_discard() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}

// ---- the two passes over one region held in registers ----------------------------------------
// A region is kRegionRows vectors per lane and row.  All of them are loaded from the stage before
// any arithmetic, and the stage's slot goes back to the producer at once; vectors past the end of
// the row read as -inf, which adds nothing to any sum and is never stored.

// Pass 1: the region's softmax sums relative to the warp's integer references (RT, RD), added to
// the running sums.  References need not be the exact maxima: any integers work as long as nothing
// overflows, and sums under different references are merged exactly later.  So only the first
// region of a unit looks for its maxima first; later ones reuse the references, and a region whose
// sums come out too large for comfort (an entry far above everything the warp has seen: rare) is
// done again after its maxima have raised the references and the running sums have moved with them
// (exact: powers of two).  The second try also serves regions with masked target entries (-inf
// logits), which the first one does not test for.
struct Pass1State {
    float RT, RD;
    LaneSums ls;
};

// The region's maxima raise the references; the running sums follow.
template <int DT, bool BONUS>
__device__ __forceinline__ void raise_references(const uint4 (&rt)[kRegionRows], const uint4 (&rd)[kRegionRows],
                                                 float c, Pass1State& s) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    float mT[kRegionRows], mD[kRegionRows];
#pragma unroll
    for (int g = 0; g < kRegionRows; ++g) {
        float v[VEC];
        E::unpack(rt[g], v);
        mT[g] = tree_max<VEC>(v);
        if (!BONUS) {
            E::unpack(rd[g], v);
            mD[g] = tree_max<VEC>(v);
        }
    }
    const float nT = fmaxf(s.RT, warp_max_ref(ref_of(tree_max<kRegionRows>(mT), c)));
    const float nD = BONUS ? kEmptyRef : fmaxf(s.RD, warp_max_ref(ref_of(tree_max<kRegionRows>(mD), c)));
    s.ls.rescale(nT - s.RT, nD - s.RD);
    s.RT = nT;
    s.RD = nD;
}

// The warp's region of a stage (st: where the region starts in the stage's target part; the draft
// part lies kStageVecs vectors further) into registers; nv = vectors of the region that exist.
template <int DT, bool BONUS>
__device__ __forceinline__ void load_region(const uint4* st, int nv, int lane, uint4 (&rt)[kRegionRows],
                                            uint4 (&rd)[kRegionRows]) {
    using E = Elem<DT>;
    if (nv == kRegionVecs) {
#pragma unroll
        for (int g = 0; g < kRegionRows; ++g) {
            rt[g] = st[g * 32 + lane];
            if (!BONUS) rd[g] = st[kStageVecs + g * 32 + lane];
        }
    } else {
#pragma unroll
        for (int g = 0; g < kRegionRows; ++g) {
            const int vi = g * 32 + lane;
            rt[g] = vi < nv ? st[vi] : E::masked();
            if (!BONUS) rd[g] = vi < nv ? st[kStageVecs + vi] : E::masked();
        }
    }
}

// Returns only when every vector of the region has arrived in this lane's registers (the value
// depends on all of them), so that the stage's slot may be overwritten afterwards.
template <bool BONUS>
__device__ __forceinline__ void await_region_registers(const uint4 (&rt)[kRegionRows], const uint4 (&rd)[kRegionRows]) {
    uint32_t dep = 0;
#pragma unroll
    for (int g = 0; g < kRegionRows; ++g) {
        dep ^= rt[g].w;
        if (!BONUS) dep ^= rd[g].w;
    }
    asm volatile("" ::"r"(dep) : "memory");
}

template <int DT, bool BONUS, bool MASKED>
__device__ __forceinline__ void region_sums_of(const uint4 (&rt)[kRegionRows], const uint4 (&rd)[kRegionRows], float c,
                                               float RT, float RD, float& sT, float& sD, float& sW) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    sT = sD = sW = 0.f;
#pragma unroll
    for (int g = 0; g < kRegionRows; ++g) {
        float tv[VEC];
        E::unpack(rt[g], tv);
        if (!BONUS) {
            float dv[VEC], pT, pD, pW;
            E::unpack(rd[g], dv);
            LaneSums::vector_pair<VEC, MASKED>(tv, dv, c, -RT, -RD, pT, pD, pW);
            sT += pT;
            sD += pD;
            sW += pW;
        } else {
            sT += LaneSums::vector_bonus<VEC>(tv, c, -RT);
        }
    }
}

// The slow way, out of line: maxima first, then the sums.  By now the stage's slot in the ring
// has been handed back, so the region is read once more from global memory (gT, gD: where it
// starts in the two rows).
template <int DT, bool BONUS>
__device__ __noinline__ Pass1State pass1_region_again(const uint4* gT, const uint4* gD, int nv, int lane, float c,
                                                      Pass1State s) {
    using E = Elem<DT>;
    uint4 rt[kRegionRows], rd[kRegionRows];
    if (nv <= 0) return s;
#pragma unroll
    for (int g = 0; g < kRegionRows; ++g) {
        const int vi = g * 32 + lane;
        const int vc = min(vi, nv - 1);       // every address formed is one of the region's own
        const uint4 a = __ldg(gT + vc);
        rt[g] = vi < nv ? a : E::masked();
        if (!BONUS) {
            const uint4 b = __ldg(gD + vc);
            rd[g] = vi < nv ? b : E::masked();
        }
    }
    raise_references<DT, BONUS>(rt, rd, c, s);
    float sT, sD, sW;
    region_sums_of<DT, BONUS, true>(rt, rd, c, s.RT, s.RD, sT, sD, sW);
    s.ls.sT += sT;
    s.ls.sD += sD;
    s.ls.w += sW;
    return s;
}

// `handed_back` is called once the region is in registers: the warp gives up its share of the slot
// then.  `again(state)` does the region the slow way (pass1_region_again) and returns the new state.
template <int DT, bool BONUS, class F, class A>
__device__ __forceinline__ void pass1_region(const uint4* st, int nv, int lane, float c, bool first, Pass1State& s,
                                             F&& handed_back, A&& again) {
    constexpr float kTooLarge = 1.152921504606846976e18f;   // 2^60
    uint4 rt[kRegionRows], rd[kRegionRows];
    load_region<DT, BONUS>(st, nv, lane, rt, rd);
    await_region_registers<BONUS>(rt, rd);
    handed_back();
    // A region cut short by the end of the slice holds -inf in place of the missing vectors, for which
    // the fast arithmetic has no test: it goes the slow way at once, like (after the vote below) a
    // region with masked target entries or with entries far above the references.
    if (nv != kRegionVecs) {
        s = again(s);
        return;
    }
    if (first) raise_references<DT, BONUS>(rt, rd, c, s);
    float sT, sD, sW;
    region_sums_of<DT, BONUS, false>(rt, rd, c, s.RT, s.RD, sT, sD, sW);
    // Too large (written so that a NaN counts as too large), or a masked target entry has turned
    // the sum of the products into a NaN: the slow way, which looks for the maxima and tests for
    // masked entries.
    if (__any_sync(0xffffffffu, !(sT < kTooLarge) || !(sD < kTooLarge) || sW != sW)) {
        s = again(s);
        return;
    }
    s.ls.sT += sT;
    s.ls.sD += sD;
    s.ls.w += sW;
}

// Pass 2 of a region held in registers: gradient out (gdst = where the region's part of the
// gradient row starts, or null) and the region's mass (sum of max(0,p-q)/tau, or of p on the
// bonus row), in every lane.  HINT: hq holds the region of the hint (the last round's gradient), and
// this lane's sum of squared differences between hint and gradient is added to herr.
template <int DT, bool BONUS, bool HINT>
__device__ __forceinline__ float pass2_region_impl(const uint4 (&rt)[kRegionRows], const uint4 (&rd)[kRegionRows], int nv,
                                                   int lane, float c, const RowConst& rc, typename Elem<DT>::type* gdst,
                                                   const uint4 (&hq)[kRegionRows], float& herr) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    float ms[kRegionRows];
#pragma unroll
    for (int g = 0; g < kRegionRows; ++g) {
        const int vi = g * 32 + lane;
        float tv[VEC], r[VEC];
        E::unpack(rt[g], tv);
        if (!BONUS) {
            float dv[VEC], gv[VEC];
            E::unpack(rd[g], dv);
            float2 acc = make_float2(0.f, 0.f);
#pragma unroll
            for (int z = 0; z < VEC; z += 2) {
                const float2 g2 = grad_elem2(make_float2(tv[z], tv[z + 1]), make_float2(dv[z], dv[z + 1]), c, rc);
                gv[z] = g2.x;
                gv[z + 1] = g2.y;
                acc = __fadd2_rn(acc, make_float2(fmaxf(-g2.x, 0.f), fmaxf(-g2.y, 0.f)));
            }
            if (gdst && vi < nv) store_streaming(gdst + (size_t)vi * VEC, E::pack(gv));
            if constexpr (HINT) {
                // distance to the hint, against the gradient before it is rounded to the output type
                if (vi < nv) {
                    float hv[VEC];
                    E::unpack(hq[g], hv);
#pragma unroll
                    for (int z = 0; z < VEC; ++z) {
                        const float dlt = hv[z] - gv[z];
                        herr = fmaf(dlt, dlt, herr);
                    }
                }
            }
            ms[g] = acc.x + acc.y;
        } else {
#pragma unroll
            for (int z = 0; z < VEC; ++z) r[z] = prob_elem(tv[z], c, rc);
            ms[g] = tree_sum<VEC>(r);
        }
    }
    float mass = tree_sum<kRegionRows>(ms);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
    return mass;
}
template <int DT, bool BONUS>
__device__ __forceinline__ float pass2_region(const uint4 (&rt)[kRegionRows], const uint4 (&rd)[kRegionRows], int nv,
                                              int lane, float c, const RowConst& rc, typename Elem<DT>::type* gdst) {
    float unused = 0.f;
    return pass2_region_impl<DT, BONUS, false>(rt, rd, nv, lane, c, rc, gdst, rt, unused);
}

// Control block of the fast path; lives in dynamic shared memory after the ring.
struct StreamShared {
    uint64_t full[kRingStages];         // stage filled by the bulk copies        (1 arrival + bytes)
    uint64_t empty[kRingStages];        // stage taken into registers by everyone (consumer warps)
    uint64_t s1_done[2];                // consumers' sums of a unit posted       (consumer warps)
    uint64_t xchg_bar[2];               // partials of every block have arrived   (1 arrival + bytes, remote)
    uint64_t rc_ready[2];               // row constants published                (1)
    uint64_t row_pub[kDoneDepth];       // statistics of the unit's row published (1)
    uint64_t s2_done[kDoneDepth];       // unit finished in this block            (consumer warps)
    uint64_t res_free[kDoneDepth];      // resolver is done with the unit         (1)
    PartialStats wpart[2][kConsumerWarps];   // the consumer warps' partials of a unit
    PartialStats xchg[2][kMaxCluster];  // written by every block of the cluster (distributed shared memory)
    PartialStats row[kDoneDepth];       // statistics of the whole row, for the row report
    RowConst rc[2];
    RowConst rc_done[kDoneDepth];       // the same, kept for the row report
    float hpart[kDoneDepth][kConsumerWarps];   // the consumer warps' shares of a unit's hint error
    int abort;                          // a bounded wait gave up somewhere in this block
};

// Units [u0, u0+n) of cluster `cid` of `G`: contiguous, sizes differ by at most one.
__device__ __host__ __forceinline__ void cluster_units(int units, int G, int cid, int& u0, int& n) {
    const int base = units / G, rem = units % G;
    n = base + (cid < rem ? 1 : 0);
    u0 = cid * base + (cid < rem ? cid : rem);
}

// The order in which a block walks the stages of its slice.  There are nst stages in every pass.
// Pass 2 of a unit needs the row constants, which take an exchange between the blocks of the
// cluster; so it is scheduled after the first L stages of pass 1 of the next unit, and it runs
// from the last stage to the first (what pass 1 fetched last is what L2 is surest to hold still):
//   S1(0)[0,nst)  then for j = 1 .. nu-1:  S1(j)[0,L)  S2(j-1)(nst,0]  S1(j)[L,nst)   then  S2(nu-1)(nst,0]
// The smaller L, the less data lies between the two passes (it has to stay in L2 meanwhile).
// (Letting the two passes alternate stage by stage was measured too: it doubles that data and is
// slower on every workload.)  The producer and every consumer warp go through the same list;
// p1(j, t0, t1, last) stands for the stages [t0,t1) of pass 1 of unit j (last: the pass is over
// afterwards), p2(j) for pass 2.
template <class P1, class P2>
__device__ __forceinline__ void walk_stages(int nu, int nst, int L, P1&& p1, P2&& p2) {
    for (int j = 0; j < nu; ++j) {
        const int head = (j == 0) ? nst : L;
        if (!p1(j, 0, head, head == nst)) return;
        if (j > 0 && !p2(j - 1)) return;
        if (head < nst && !p1(j, head, nst, true)) return;
    }
    if (nu > 0) p2(nu - 1);
}

// ---- fast path -----------------------------------------------------------------------------
// lag_stages: stages of pass 1 of the next unit that go before pass 2 of a unit.
// prefetch: non-zero lets the producer ask L2 for the next unit's pass-1 stages during pass 2.
// ENS: the units are those of the ensemble feedback (see UnitRef); nothing is verified or drawn.
// STATS: pass 1 only -- row constants, losses and rejection tests of every row; no gradient, no
// masses, no draw (the error-position feedback finishes the one row it needs in a kernel of its own).
// HINT: pass 2 also reads the hint of the optimistic update (the last round's gradient) and sums its
// squared distance to this round's gradient per row.
template <int DT, bool ENS, bool STATS = false, bool HINT = false>
__global__ void __launch_bounds__(kStreamThreads, 1)
sd_stream_kernel(const __grid_constant__ Params P, const int lag_stages, const int prefetch) {
    using E = Elem<DT>;
    using ET = typename E::type;
    constexpr int VEC = E::VEC;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;
    constexpr int kRing = RingStages<DT>::value;
    StreamShared& sh = *reinterpret_cast<StreamShared*>(dyn_smem + (size_t)kRing * kStageBytes);

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
    const int regions_row = (NV + kRegionVecs - 1) / kRegionVecs;   // = P.NR
    const int regions_blk = (regions_row + C - 1) / C;
    const int r0 = rank * regions_blk;            // first region of this block's slice
    const int nr = max(0, min(regions_row - r0, regions_blk));      // regions of the slice
    const int vb0 = r0 * kRegionVecs;             // first vector of the slice
    const int nvb = max(0, min(NV - vb0, nr * kRegionVecs));        // vectors of the slice
    const int nst = (nr + kConsumerWarps - 1) / kConsumerWarps;     // stages of a pass
    // lag_stages = -2: every other cluster takes all of the next unit's pass 1 first, the rest none of it,
    // so that half of the GPU reads from HBM while the other half works from L2
    const int L = lag_stages == -2 ? ((cid & 1) ? nst : 0) : min(max(lag_stages, 0), nst);
    const WaitCtx wc{&sh.abort, P.wait_polls};

    if (tid == 0) {
        for (int s = 0; s < kRing; ++s) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], kConsumerWarps);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(&sh.s1_done[s], kConsumerWarps);
            mbar_init(&sh.xchg_bar[s], 1);
            mbar_init(&sh.rc_ready[s], 1);
        }
        for (int s = 0; s < kDoneDepth; ++s) {
            mbar_init(&sh.row_pub[s], 1);
            mbar_init(&sh.s2_done[s], kConsumerWarps);
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
            if (C > 1 && lane == 0) mbar_expect_tx(&sh.xchg_bar[par], (uint32_t)C * (uint32_t)sizeof(PartialStats));
            if (!mbar_wait(&sh.s1_done[par], ph, wc)) break;
            // the block's partial from its warps' partials, then (in a cluster of several blocks) one
            // copy to every block of the cluster
            PartialStats row = warp_merge_lanes(lane < kConsumerWarps ? sh.wpart[par][lane] : empty_partial());
            if (C > 1) {
                if (lane < C) {
                    uint64_t refs;
                    memcpy(&refs, &row.RT, 8);
                    PartialStats* dst = &sh.xchg[par][rank];
                    st_async_remote(dst, refs, (uint64_t)__double_as_longlong(row.sT), &sh.xchg_bar[par], (uint32_t)lane);
                    st_async_remote(&dst->sD, (uint64_t)__double_as_longlong(row.sD), (uint64_t)__double_as_longlong(row.w),
                                    &sh.xchg_bar[par], (uint32_t)lane);
                }
                if (!mbar_wait_cluster(&sh.xchg_bar[par], ph, wc)) break;
                row = warp_merge_lanes(lane < C ? sh.xchg[par][lane] : empty_partial());
            }
            const RowConst rcw = row_constants(P, bonus, row);
            if (lane == 0) {
                sh.rc[par] = rcw;
                mbar_arrive(&sh.rc_ready[par]);
                // for the row report by the resolver: wait until it is done with the slot's last use
                bool ok = true;
                if (j >= kDoneDepth)
                    ok = mbar_wait_thread<false>(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, wc);
                if (ok) {
                    sh.row[dslot] = row;
                    sh.rc_done[dslot] = rcw;
                    mbar_arrive(&sh.row_pub[dslot]);
                }
            }
            if (__any_sync(0xffffffffu, sh.abort)) break;
        }
    } else if (warp == kResolverWarp) {
        // ---- resolver: row reports, tickets; the sequence's last tickets draw the token
        int seg = 0;                               // units of the current sequence finished so far
        for (int j = 0; j < nu; ++j) {
            const int unit = u0 + j * ustep;
            const int dslot = j % kDoneDepth;
            const bool reports = (j % C == rank);   // the blocks of the cluster take turns
            const uint32_t dph = (uint32_t)(j / kDoneDepth) & 1u;
            if constexpr (ENS) {
                if (!mbar_wait_sleepy<200>(&sh.row_pub[dslot], dph, wc)) break;
                if (reports && lane == 0) finish_row_ensemble(P, unit_ref<true>(P, unit), sh.row[dslot]);
                if (!mbar_wait_sleepy<200>(&sh.s2_done[dslot], dph, wc)) break;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
                continue;
            }
            const int b = unit / K1, i = unit - b * K1;
            const bool bonus = (i == P.k);
            AcceptOperands aop;
            aop.valid = false;
            if (reports && lane == 0 && !bonus) aop = load_accept_operands<DT>(P, b, i);
            // the row report needs pass 1 only: it runs while the consumers are in pass 2
            if (!mbar_wait_sleepy<200>(&sh.row_pub[dslot], dph, wc)) break;
            if (reports && lane == 0) finish_row(P, b, i, sh.row[dslot], sh.rc_done[dslot], aop);
            if (!mbar_wait_sleepy<200>(&sh.s2_done[dslot], dph, wc)) break;
            __syncwarp();
            if constexpr (STATS) {
                if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
                continue;
            }
            if constexpr (HINT) {
                // this block's share of the row's hint error: the warps' shares in their order, in fp64
                double hp = (lane < kConsumerWarps) ? (double)sh.hpart[dslot][lane] : 0.0;
                hp = warp_sum(hp);
                if (lane == 0 && !bonus) P.hint_part[(size_t)unit * kMaxCluster + rank] = hp;
            }
            ++seg;
            const bool leaves = (i == P.k) || (j == nu - 1);   // last unit of the sequence in this cluster
            if (leaves) {
                int last = 0;
                if (lane == 0) last = take_tickets(P, b, (uint32_t)seg) ? 1 : 0;
                last = __shfl_sync(0xffffffffu, last, 0);
                if (last) resolve_sequence<DT, true>(P, b);
                seg = 0;
                __syncwarp();
            }
            if (lane == 0) mbar_arrive(&sh.res_free[dslot]);
        }
    } else if (warp == kProducerWarp) {
        // ---- producer: two threads fetch the stages of the walk, in order, into the ring -- the first
        // arms the stage's barrier and copies the target part, the second copies the draft part (one
        // thread issuing both copies one after the other gets three quarters of the bytes per clock)
        if (lane < 2 && nst > 0) {
            const uint64_t keep = policy_keep(), discard = policy_discard();
            int ni = 0, slot = 0;                  // stages issued so far; slot of the next one
            uint32_t epar = 1;                     // parity to wait for on empty[slot]: that of its previous use
            bool ok = true;
            auto issue = [&](const UnitRef& ur, int t, uint64_t pol) {
                // (each of the two threads waits for the slot itself: a word passed from one to the other
                // costs the stage's copies a few hundred cycles of head start, 6 % on the largest workload.
                // Should only one of them give up, the other's copy lands during the pause before the block
                // exits, or the wait for a half-armed stage below runs into its time limit.)
                if (ni >= kRing && !mbar_wait_thread<false>(&sh.empty[slot], epar, wc)) { ok = false; return; }
                const int v0 = t * kStageVecs;     // first vector of the stage within the slice
                const uint32_t bytes = (uint32_t)min(kStageVecs, nvb - v0) * 16u;
                const size_t off = (size_t)(vb0 + v0) * VEC;
                unsigned char* dst = ring + (size_t)slot * kStageBytes;
#ifdef SD_BOUNDS_CHECK
                // a copy that fails its check is not issued; its bytes are counted on the stage's barrier
                // by hand instead, so that nobody waits for them (the stage then holds what it held before)
                const long long rowsT = (long long)P.B * (P.k + 1), rowsD = (long long)P.B * P.k;
                const bool okc = SD_IN(off + bytes / sizeof(ET) - 1, P.V, lane == 0 ? 10 : 11) &&
                                 (lane == 0 ? SD_IN(ur.t_row, rowsT, 10) : SD_IN(ur.d_row, rowsD, 11));
                if (!okc) {
                    if (lane == 0) mbar_expect_tx(&sh.full[slot], ur.bonus ? bytes : 2u * bytes);
                    if (lane == 0 || !ur.bonus) mbar_complete_tx(&sh.full[slot], bytes);
                } else
#endif
                if (lane == 0) {
                    mbar_expect_tx(&sh.full[slot], ur.bonus ? bytes : 2u * bytes);
                    bulk_load(dst, reinterpret_cast<const ET*>(P.T) + ur.t_row * P.V + off, bytes, &sh.full[slot], pol);
                } else if (!ur.bonus) {
                    // (its bytes may land before the barrier is armed: the count then goes below zero
                    // for a moment, and the phase cannot end before the first thread's arrival)
                    bulk_load(dst + kStageRowBytes,
                              reinterpret_cast<const ET*>(ENS ? P.Dn[ur.n] : P.D) + ur.d_row * P.V + off, bytes,
                              &sh.full[slot], pol);
                }
                ++ni;
                if (++slot == kRing) { slot = 0; epar ^= 1u; }
            };
            walk_stages(nu, nst, L,
                [&](int j, int t0, int t1, bool) {
                    const UnitRef ur = unit_ref<ENS>(P, u0 + j * ustep);
                    for (int t = t0; t < t1 && ok; ++t) issue(ur, t, STATS ? discard : keep);
                    return ok;
                },
                [&](int j) {
                    if constexpr (!STATS) {
                        const UnitRef ur = unit_ref<ENS>(P, u0 + j * ustep);
                        // Optionally each pass-2 stage issued also asks L2 to fetch one stage of pass 1 of
                        // the next unit, which spreads the HBM reads over the time the consumers spend
                        // in pass 2 (it pays when the row pairs in flight leave room in L2 for it).
                        const bool ahead = prefetch != 0 && j + 1 < nu;
                        UnitRef nx = ur;
                        if (ahead) nx = unit_ref<ENS>(P, u0 + (j + 1) * ustep);
                        for (int t = nst - 1; t >= 0 && ok; --t) {
                            issue(ur, t, discard);
                            const int tp = L + (nst - 1 - t);
                            if (ahead && ok && tp < nst) {
                                const int v0 = tp * kStageVecs;
                                const uint32_t bytes = (uint32_t)min(kStageVecs, nvb - v0) * 16u;
                                const size_t off = (size_t)(vb0 + v0) * VEC;
                                if (lane == 0)
                                    bulk_prefetch_l2(reinterpret_cast<const ET*>(P.T) + nx.t_row * P.V + off, bytes, keep);
                                else if (!nx.bonus)
                                    bulk_prefetch_l2(reinterpret_cast<const ET*>(ENS ? P.Dn[nx.n] : P.D) + nx.d_row * P.V + off, bytes, keep);
                            }
                        }
                    }
                    return ok;
                });
            // leaving early: no copy may still be in flight when the block returns
            if (!ok && lane == 0) {
                const long long t0 = clock64();
                for (int i = max(0, ni - kRing); i < ni; ++i) {
                    const uint32_t par = (uint32_t)(i / kRing) & 1u;
                    for (uint32_t it = 0; it < kWaitLimit && !mbar_try_wait(&sh.full[i % kRing], par); ++it)
                        if (clock64() - t0 > kWaitCycles) break;
                }
            }
        }
    } else if (warp >= kFirstConsumerWarp) {
        // ---- consumers: warp cw owns region cw of every stage; a region is a sampling region.
        const int cw = warp - kFirstConsumerWarp;
        const int rv0 = cw * kRegionVecs;          // where my region starts within a stage
        int slot = 0;                              // ring slot of the next stage and the parity of its full barrier
        uint32_t fpar = 0;
        bool ok = true;
        // The region is in registers: hand the warp's share of the slot back.  (Every lane's loads
        // from the slot have returned their values before the arrival.)
        // Afterwards a look (no waiting) at the barrier of the next stage: its answer is there long
        // before the arithmetic on this region is over, and when it says "full" -- the usual case --
        // the next visit starts without the round trip of a wait.
        bool next_full = false;
        auto hand_back = [&]() {
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.empty[slot]);
            if (++slot == kRing) { slot = 0; fpar ^= 1u; }
            next_full = mbar_test(&sh.full[slot], fpar);
        };
        auto await_stage = [&]() {
            if (__all_sync(0xffffffffu, next_full ? 1 : 0)) return true;
            return mbar_wait(&sh.full[slot], fpar, wc);
        };
        Pass1State ps;
        ps.RT = ps.RD = kEmptyRef;
        ps.ls.init();
        auto vectors_of = [&](int t) { return max(0, min(kRegionVecs, nvb - t * kStageVecs - rv0)); };   // of my region of stage t
        auto run_pass1 = [&](int j, int t0, int t1, bool last) {
            const UnitRef ur = unit_ref<ENS>(P, u0 + j * ustep);
            const bool bonus = ur.bonus;
            for (int t = t0; t < t1; ++t) {
                if (!await_stage()) { ok = false; return false; }
                const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes) + rv0;
                const int nv = vectors_of(t);
                if (nv == 0) { hand_back(); continue; }
                // where the region lies in global memory: only the rare second try of a region reads it there
                auto again = [&](Pass1State s0) {
                    const size_t voff = (size_t)vb0 + rv0 + (size_t)t * kStageVecs;
                    if (!SD_IN((voff + nv) * VEC - 1, P.V, 14)) return s0;
                    const uint4* gT = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.T) + ur.t_row * P.V) + voff;
                    const uint4* gD = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(ENS ? P.Dn[ur.n] : P.D) + ur.d_row * P.V) + voff;
                    return bonus ? pass1_region_again<DT, true>(gT, gD, nv, lane, P.c, s0)
                                 : pass1_region_again<DT, false>(gT, gD, nv, lane, P.c, s0);
                };
                if (bonus) pass1_region<DT, true>(st, nv, lane, P.c, t == 0, ps, hand_back, again);
                else       pass1_region<DT, false>(st, nv, lane, P.c, t == 0, ps, hand_back, again);
            }
            if (last) {
                // pass 1 of the unit is over: the warp's partial for the statistics warp
                const PartialStats part = warp_sum_lanes(ps.ls, ps.RT, ps.RD);
                if (lane == 0) {
                    sh.wpart[j & 1][cw] = part;
                    mbar_arrive(&sh.s1_done[j & 1]);
                }
                ps.RT = ps.RD = kEmptyRef;
                ps.ls.init();
                if constexpr (STATS) {
                    // nothing else to do for the unit but to report it finished -- after its row
                    // constants are out, as in the full walk: the statistics warp is then done with
                    // the partials of the unit, whose slots the unit after next reuses
                    const int dslot = j % kDoneDepth;
                    if (!mbar_wait(&sh.rc_ready[j & 1], (uint32_t)(j >> 1) & 1u, wc)) { ok = false; return false; }
                    if (j >= kDoneDepth &&
                        !mbar_wait(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, wc)) { ok = false; return false; }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
                }
            }
            return true;
        };
        auto run_pass2 = [&](int j) {
            if constexpr (STATS) return true;
            const int unit = u0 + j * ustep;
            const UnitRef ur = unit_ref<ENS>(P, unit);
            const bool bonus = ur.bonus;
            const int dslot = j % kDoneDepth;
            if (!mbar_wait(&sh.rc_ready[j & 1], (uint32_t)(j >> 1) & 1u, wc)) { ok = false; return false; }
            const RowConst rc = sh.rc[j & 1];
            void* const gbase = ENS ? P.Gn[ur.n] : P.grad;
            ET* Grow = (gbase && !bonus) ? reinterpret_cast<ET*>(gbase) + ur.d_row * P.V + (size_t)(vb0 + rv0) * VEC : nullptr;
            float* rsum = ENS ? nullptr : P.region_sums + (size_t)unit * P.NR + r0 + cw;
            const uint4* Hrow = nullptr;
            if constexpr (HINT)
                Hrow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.hint) + ur.d_row * P.V) + vb0 + rv0;
            float herr = 0.f;
            for (int t = nst - 1; t >= 0; --t) {
                const int nv = vectors_of(t);
                // the hint does not go through the ring: each lane asks for its vectors before it waits
                // for the stage, and they are there when the gradient is
#ifdef SD_BOUNDS_CHECK
                const size_t vfirst = (size_t)vb0 + rv0 + (size_t)t * kStageVecs;   // first vector of my region in the row
                const bool in_row = nv == 0 || SD_IN((vfirst + nv) * VEC - 1, P.V, 12);
#else
                constexpr bool in_row = true;
#endif
                uint4 hq[kRegionRows];
                if constexpr (HINT) {
#pragma unroll
                    for (int g = 0; g < kRegionRows; ++g)
                        hq[g] = (!bonus && in_row && g * 32 + lane < nv) ? __ldcs(Hrow + (size_t)t * kStageVecs + g * 32 + lane)
                                                               : make_uint4(0u, 0u, 0u, 0u);
                }
                if (!await_stage()) { ok = false; return false; }
                const uint4* st = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes) + rv0;
                if (nv == 0) { hand_back(); continue; }
                uint4 rt[kRegionRows], rd[kRegionRows];
                if (bonus) { load_region<DT, true>(st, nv, lane, rt, rd); await_region_registers<true>(rt, rd); }
                else       { load_region<DT, false>(st, nv, lane, rt, rd); await_region_registers<false>(rt, rd); }
                hand_back();
                float mass;
                if constexpr (HINT) {
                    mass = bonus ? pass2_region<DT, true>(rt, rd, nv, lane, P.c, rc, nullptr)
                                 : pass2_region_impl<DT, false, true>(rt, rd, nv, lane, P.c, rc,
                                                                      (Grow && in_row) ? Grow + (size_t)t * kStageVecs * VEC : nullptr,
                                                                      hq, herr);
                } else {
                    mass = bonus ? pass2_region<DT, true>(rt, rd, nv, lane, P.c, rc, nullptr)
                                 : pass2_region<DT, false>(rt, rd, nv, lane, P.c, rc,
                                                           (Grow && in_row) ? Grow + (size_t)t * kStageVecs * VEC : nullptr);
                }
                if (!ENS && lane == 0 && SD_IN(r0 + cw + t * kConsumerWarps, P.NR, 13)) rsum[t * kConsumerWarps] = mass;
            }
            if constexpr (HINT) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) herr += __shfl_xor_sync(0xffffffffu, herr, off);
            }
            // the resolver's slot of unit j-4 must be free again before this unit is reported done
            if (j >= kDoneDepth &&
                !mbar_wait(&sh.res_free[dslot], (uint32_t)(j / kDoneDepth - 1) & 1u, wc)) { ok = false; return false; }
            __syncwarp();
            if (lane == 0) {
                if constexpr (HINT) sh.hpart[dslot][cw] = herr;
                mbar_arrive(&sh.s2_done[dslot]);
            }
            return true;
        };
        walk_stages(nu, nst, L, run_pass1, run_pass2);
    }

    __syncthreads();
    if (sh.abort) {
        // a wait gave up: say so in every sequence this cluster has a unit of, and in every
        // sequence resolved from now on
        if (tid == 0) atomicExch(P.sticky, 1u);
        if (P.status)
            for (int j = tid; j < nu; j += kStreamThreads) atomicOr(P.status + unit_ref<ENS>(P, u0 + j * ustep).b, kStatusTimeout);
        // whatever another block of the cluster has sent to this one's shared memory meanwhile has
        // had time to land before the block goes away
        for (int i = 0; i < 20; ++i) __nanosleep(1000);
    }
    // no block leaves while another may still write to its shared memory
    cluster.sync();
}

// ---- generic path --------------------------------------------------------------------------
struct GenericShared {
    PartialStats warp_part[kGenericWarps];
    float hpart[kGenericWarps];
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
    float herr = 0.f;
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
                    if (P.hint) {
                        const float dlt = E::load(P.hint, offD + v) - g;
                        herr = fmaf(dlt, dlt, herr);
                    }
                    if (P.grad && SD_IN(offD + v, (long long)P.B * P.k * P.V, 31)) E::store(P.grad, offD + v, g);
                } else {
                    mass += prob_elem(t, P.c, rc);
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
        if (lane == 0 && SD_IN((long long)unit * P.NR + q, (long long)P.B * (P.k + 1) * P.NR, 32)) rsum[q] = mass;
    }

    if (P.hint) {
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) herr += __shfl_xor_sync(0xffffffffu, herr, off);
        if (lane == 0) sh.hpart[warp] = herr;
    }
    // the block that takes the sequence's last ticket resolves it
    __syncthreads();
    if (tid == 0 && P.hint && !bonus) {
        double e = 0.0;
        for (int w = 0; w < kGenericWarps; ++w) e += (double)sh.hpart[w];
        P.hint_part[(size_t)unit * kMaxCluster] = e;
    }
    if (tid == 0) sh.last = take_tickets(P, b, 1u) ? 1 : 0;
    __syncthreads();
    if (sh.last && warp == 0) resolve_sequence<DT, false>(P, b);
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
