// The two kernels of the verify-and-feedback step.
//
//   sd_stream_kernel   fast path.  A persistent kernel of thread-block clusters.  A cluster takes a
//                      contiguous range of (sequence, row) units, one after the other; each block
//                      of the cluster owns a contiguous slice of the vocabulary, and each of its
//                      16 consumer warps a contiguous part of that slice (a sampling region).
//                      A slice is streamed through a ring of small shared-memory stages twice:
//                      pass 1 (maxima, then softmax sums relative to integer references) reads it
//                      from HBM, pass 2 (gradient out, residual mass) reads it again a few
//                      microseconds later, when it is still in L2, so HBM sees each logit once.
//                      Inside a block the warps are specialised:
//                        producer   its lanes issue the bulk asynchronous copies (cp.async.bulk +
//                                   mbarrier) of both passes in consumption order, running ahead
//                                   as far as the ring allows, so memory never waits for arithmetic;
//                        consumers  each works through the stages of its own region and hands
//                                   them back; warps meet only once per unit and pass;
//                        statistics adds up the consumers' sums, exchanges the block's partial
//                                   with the other blocks of the cluster through distributed
//                                   shared memory (remote stores + remote mbarrier arrivals, no
//                                   cluster-wide barrier) and publishes the row constants;
//                        resolver   turns the lanes' residual masses into region sums, reports
//                                   rows (loss, rejection test), takes the sequence's tickets when
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
// A row is cut into sampling regions of `per` 16-byte vectors (per = 32*m, m >= 4).  Block r of
// a cluster owns the 16 regions [16r, 16r+16) of every row it works on, one per consumer warp.
// The block's slice is streamed in stages of 128 vectors (2 KiB) per row, so group g of 32 vectors
// of the slice lies in stage g/4, and a stage is used by one consumer warp or by two neighbours.
constexpr int kConsumerWarps = 16;
constexpr int kStageGroups = 4;                               // groups of 32 vectors in a stage
constexpr int kStageVecs = 32 * kStageGroups;                 // vectors of one row in a stage
constexpr int kStageRowBytes = kStageVecs * 16;               // 2 KiB of one row
constexpr int kStageBytes = 2 * kStageRowBytes;               // target part + draft part
constexpr int kRingSlots = 48;                                // 192 KiB
constexpr int kDoneDepth = 4;                                 // units the resolver may lag behind
constexpr int kProducerWarp = 0, kStatsWarp = 1, kResolverWarp = 2, kFirstConsumerWarp = 3;
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
__device__ __forceinline__ void mbar_arrive_n(uint64_t* bar, uint32_t n) {
    asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(n) : "memory");
}
__device__ __forceinline__ uint32_t ld_acquire_shared(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.cta.shared::cta.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
    return v;
}
__device__ __forceinline__ void st_release_shared(uint32_t* p, uint32_t v) {
    asm volatile("st.release.cta.shared::cta.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
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
template <bool CLUSTER>
__device__ __forceinline__ bool mbar_wait_thread(uint64_t* bar, uint32_t parity, volatile int* abort) {
    long long t0 = 0;
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (CLUSTER ? mbar_try_wait_cluster(bar, parity) : mbar_try_wait(bar, parity)) return true;
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
    return __all_sync(0xffffffffu, mbar_wait_thread<true>(bar, parity, abort) ? 1 : 0) != 0;
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
// L2 policies: keep (a line that will be read again shortly) and drop (a line nobody reads again).
__device__ __forceinline__ uint64_t policy_keep() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t policy_drop() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
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

// Control block of the fast path; lives in dynamic shared memory after the ring.
struct StreamShared {
    uint64_t full[kRingSlots];          // stage filled by the bulk copies        (1 arrival + bytes)
    uint64_t empty[kRingSlots];         // stage handed back                      (2: its one or two users)
    uint32_t issued[kRingSlots];        // uses of the slot whose copies have been issued so far
    uint64_t s1_done[2];                // consumers' sums of a unit posted       (consumer warps)
    uint64_t xchg_bar[2];               // partials of every block have arrived   (cluster size, remote)
    uint64_t rc_ready[2];               // row constants published                (1)
    uint64_t s2_done[kDoneDepth];       // unit finished in this block            (consumer warps + 1)
    uint64_t res_free[kDoneDepth];      // resolver is done with the unit         (1)
    float lane_sums[2][3][kConsumerWarps][33];        // sT, sD, w of every consumer lane (33: no bank conflicts)
    float warp_ref[2][kConsumerWarps][2];             // RT, RD each consumer warp used
    float lane_mass[kDoneDepth][kConsumerWarps][33];  // residual / bonus mass of every consumer lane
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

    const int per = P.RE / VEC;                   // vectors per sampling region
    const int m = per >> 5;                       // groups of 32 vectors per region
    const int NV = P.V / VEC;                     // vectors per row
    const int vb0 = rank * kConsumerWarps * per;  // first vector of this block's slice
    const int nvb = max(0, min(NV - vb0, kConsumerWarps * per));
    const int ns = (nvb + kStageVecs - 1) / kStageVecs;   // stages of a pass
    const int tg = (nvb + 31) >> 5;                       // groups of the slice
    const PassOrder order{nu, lag};
    volatile int* abort = &sh.abort;

    if (tid == 0) {
        for (int s = 0; s < R; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 2); sh.issued[s] = 0; }
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

    if (warp == kProducerWarp) {
        // ---- producer: lane l issues the copies of the stages that go to ring slots l and l+32,
        // in the order of their sequence numbers q (stage s of pass p has q = p*ns + s, slot q % R)
        const uint64_t keep = policy_keep(), drop = policy_drop();
        const long long total = (long long)order.count() * ns;   // stages this block streams
        bool ok = true;
        long long q_last = -1;
        long long qa = lane, qb = (lane + 32 < R) ? (long long)(lane + 32) : total;
        while (ok) {
            const long long q = qa < qb ? qa : qb;
            if (q >= total) break;
            if (q == qa) qa += R; else qb += R;
            const int slot = (int)(q % R);
            const uint32_t use = (uint32_t)(q / R);
            const int p = (int)(q / ns), s = (int)(q - (long long)p * ns);
            int j, kind;
            order.decode(p, j, kind);
            const int unit = u0 + j;
            const int b = unit / K1, i = unit - b * K1;
            const bool bonus = (i == P.k);
            if (use > 0 && !mbar_wait_thread<false>(&sh.empty[slot], (use - 1) & 1u, abort)) { ok = false; break; }
            const int v0 = s * kStageVecs;
            const uint32_t bytes = (uint32_t)min(kStageVecs, nvb - v0) * 16u;
            const ET* Tsrc = reinterpret_cast<const ET*>(P.T) + (size_t)unit * P.V + (size_t)(vb0 + v0) * VEC;
            unsigned char* dst = ring + (size_t)slot * kStageBytes;
            const uint64_t pol = kind == 0 ? keep : drop;
            mbar_expect_tx(&sh.full[slot], bonus ? bytes : 2u * bytes);
            bulk_load(dst, Tsrc, bytes, &sh.full[slot], pol);
            if (!bonus) {
                const ET* Dsrc = reinterpret_cast<const ET*>(P.D) + (size_t)(b * P.k + i) * P.V + (size_t)(vb0 + v0) * VEC;
                bulk_load(dst + kStageRowBytes, Dsrc, bytes, &sh.full[slot], pol);
            }
            st_release_shared(&sh.issued[slot], use + 1u);
            q_last = q;
        }
        if (__any_sync(0xffffffffu, !ok || *abort)) {
            // giving up: no copy may still be in flight when the block returns
            for (int slot = lane; slot < R; slot += 32) {
                long long q = -1;                       // last use this lane issued into the slot
                for (long long t = slot; t <= q_last; t += R) q = t;
                if (q >= 0) {
                    const uint32_t par = (uint32_t)(q / R) & 1u;
                    for (uint32_t it = 0; it < kWaitLimit && !mbar_try_wait(&sh.full[slot], par); ++it) {}
                }
            }
        }
    } else if (warp == kStatsWarp) {
        // ---- statistics: block partial -> cluster exchange -> row constants
        for (int j = 0; j < nu; ++j) {
            const int unit = u0 + j;
            const bool bonus = (unit % K1 == P.k);
            const int par = j & 1;
            const uint32_t ph = (uint32_t)(j >> 1) & 1u;
            const int dslot = j % kDoneDepth;
            if (!mbar_wait(&sh.s1_done[par], ph, abort)) break;
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
        // ---- resolver: region sums, row reports, tickets; the sequence's last tickets draw the token
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
            if (!mbar_wait(&sh.s2_done[dslot], (uint32_t)(j / kDoneDepth) & 1u, abort)) break;
            // mass of this block's 16 regions of the row: lane l adds up half of warp l%16's lanes
            {
                const int w = lane & 15, h0 = (lane >> 4) * 16;
                float ms = 0.f;
#pragma unroll
                for (int l = 0; l < 16; ++l) ms += sh.lane_mass[dslot][w][h0 + l];
                ms += __shfl_xor_sync(0xffffffffu, ms, 16);
                const int region = rank * kConsumerWarps + w;
                if (lane < kConsumerWarps && region < P.NR) P.region_sums[(size_t)unit * P.NR + region] = ms;
            }
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
        // ---- consumers: warp cw owns region 16*rank + cw of every row: groups [g0, g0+ng) of the slice
        const int cw = warp - kFirstConsumerWarp;
        const int g0 = cw * m;
        const int ng = max(0, min(m, tg - g0));
        const int s_first = g0 / kStageGroups, s_last = (g0 + ng - 1) / kStageGroups;   // stages of the region
        // a stage shared with the neighbouring warp is handed back by both, each counting once
        const uint32_t w_first = (g0 % kStageGroups != 0) ? 1u : 2u;
        const uint32_t w_last = ((g0 + ng) % kStageGroups != 0 && g0 + ng < tg) ? 1u : 2u;
        auto slot_of = [&](int p, int s, uint32_t& use) -> int {
            const long long q = (long long)p * ns + s;
            use = (uint32_t)(q / R);
            return (int)(q % R);
        };
        // Wait for use `use` of a slot.  Consumer warps run up to two passes apart, more than the
        // ring holds, so the parity of the barrier alone could be taken for that of an older use:
        // first wait until the copies of this very use have been issued (which happens only after
        // the previous use was handed back), then for them to land.
        auto wait_stage = [&](int slot, uint32_t use) -> bool {
            bool seen = false;
            long long t0 = 0;
            for (uint32_t it = 0; it < kWaitLimit; ++it) {
                if (ld_acquire_shared(&sh.issued[slot]) > use) { seen = true; break; }
                if ((it & 63u) == 63u) {
                    if (*abort) break;
                    const long long now = clock64();
                    if (t0 == 0) t0 = now;
                    else if (now - t0 > kWaitCycles) break;
                }
            }
            if (!seen) *abort = 1;
            if (!__all_sync(0xffffffffu, seen ? 1 : 0)) return false;
            return mbar_wait(&sh.full[slot], use & 1u, abort);
        };
        auto release = [&](int p, int s) {
            uint32_t use;
            const int slot = slot_of(p, s, use);
            uint32_t n = 2u;
            if (s == s_first && s == s_last) n = (w_first == 1u || w_last == 1u) ? 1u : 2u;
            else if (s == s_first) n = w_first;
            else if (s == s_last) n = w_last;
            mbar_arrive_n(&sh.empty[slot], n);
        };
        bool ok = true;
        for (int j = 0; j < nu + lag && ok; ++j) {
            if (j < nu) {
                // pass 1 of unit j.  Sweep A: the region's maxima; sweep B: sums relative to them.
                const bool bonus = ((u0 + j) % K1 == P.k);
                const int p = order.index_s1(j);
                float mT = -3.402823466e+38f, mD = -3.402823466e+38f;
                int waited = -1;
                for (int t = 0; t < ng; ++t) {
                    const int g = g0 + t, st = g / kStageGroups;
                    uint32_t use;
                    const int slot = slot_of(p, st, use);
                    if (st > waited) {
                        if (!wait_stage(slot, use)) { ok = false; break; }
                        waited = st;
                    }
                    const int vi = (g % kStageGroups) * 32 + lane;
                    if (g * 32 + lane < nvb) {
                        const uint4* sT = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
                        float tv[VEC];
                        E::unpack(sT[vi], tv);
                        mT = fmaxf(mT, tree_max<VEC>(tv));
                        if (!bonus) {
                            float dv[VEC];
                            E::unpack(sT[kStageVecs + vi], dv);
                            mD = fmaxf(mD, tree_max<VEC>(dv));
                        }
                    }
                }
                if (!ok) break;
                const float RT = warp_max_ref(ref_of(mT, P.c));
                const float RD = bonus ? kEmptyRef : warp_max_ref(ref_of(mD, P.c));
                LaneSums ls;
                ls.init();
                for (int t = 0; t < ng; ++t) {
                    const int g = g0 + t;
                    uint32_t use;
                    const int slot = slot_of(p, g / kStageGroups, use);
                    const int vi = (g % kStageGroups) * 32 + lane;
                    if (g * 32 + lane < nvb) {
                        const uint4* sT = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
                        float tv[VEC];
                        E::unpack(sT[vi], tv);
                        if (!bonus) {
                            float dv[VEC];
                            E::unpack(sT[kStageVecs + vi], dv);
                            ls.template add_pair<VEC>(tv, dv, P.c, -RT, -RD);
                        } else {
                            ls.template add_bonus<VEC>(tv, P.c, -RT);
                        }
                    }
                }
                const int parj = j & 1;
                sh.lane_sums[parj][0][cw][lane] = ls.sT;
                sh.lane_sums[parj][1][cw][lane] = ls.sD;
                sh.lane_sums[parj][2][cw][lane] = ls.w;
                if (lane == 0) { sh.warp_ref[parj][cw][0] = RT; sh.warp_ref[parj][cw][1] = RD; }
                __syncwarp();
                if (lane == 0) {
                    if (ng > 0)
                        for (int s = s_first; s <= s_last; ++s) release(p, s);
                    mbar_arrive(&sh.s1_done[parj]);
                }
            }
            if (j >= lag) {
                // pass 2 of unit j-lag
                const int jj = j - lag;
                const int unit = u0 + jj;
                const int b = unit / K1, i = unit - b * K1;
                const bool bonus = (i == P.k);
                const int dslot = jj % kDoneDepth;
                const int p = order.index_s2(jj);
                if (!mbar_wait(&sh.rc_ready[jj & 1], (uint32_t)(jj >> 1) & 1u, abort)) { ok = false; break; }
                const RowConst rc = sh.rc[jj & 1];
                ET* Grow = (P.grad && !bonus)
                               ? reinterpret_cast<ET*>(P.grad) + (size_t)(b * P.k + i) * P.V + (size_t)vb0 * VEC
                               : nullptr;
                float mass = 0.f;
                int cur = -1;         // stage being worked on
                for (int t = 0; t < ng; ++t) {
                    const int g = g0 + t, st = g / kStageGroups;
                    uint32_t use;
                    const int slot = slot_of(p, st, use);
                    if (st != cur) {
                        if (cur >= 0) {
                            __syncwarp();
                            if (lane == 0) release(p, cur);
                        }
                        if (!wait_stage(slot, use)) { ok = false; break; }
                        cur = st;
                    }
                    const int vi = (g % kStageGroups) * 32 + lane;
                    if (g * 32 + lane < nvb) {
                        const uint4* sT = reinterpret_cast<const uint4*>(ring + (size_t)slot * kStageBytes);
                        float tv[VEC], r[VEC];
                        E::unpack(sT[vi], tv);
                        if (!bonus) {
                            float dv[VEC], gv[VEC];
                            E::unpack(sT[kStageVecs + vi], dv);
#pragma unroll
                            for (int z = 0; z < VEC; ++z) {
                                gv[z] = grad_elem(tv[z], dv[z], P.c, rc);
                                r[z] = fmaxf(-gv[z], 0.f);
                            }
                            if (Grow) store_streaming(Grow + (size_t)(g * 32 + lane) * VEC, E::pack(gv));
                        } else {
#pragma unroll
                            for (int z = 0; z < VEC; ++z) r[z] = prob_elem(tv[z], P.c, rc);
                        }
                        mass += tree_sum<VEC>(r);
                    }
                }
                if (!ok) break;
                __syncwarp();
                if (lane == 0 && cur >= 0) release(p, cur);
                // the resolver must be done with the slot's last use before the masses are replaced
                if (jj >= kDoneDepth &&
                    !mbar_wait(&sh.res_free[dslot], (uint32_t)(jj / kDoneDepth - 1) & 1u, abort)) { ok = false; break; }
                sh.lane_mass[dslot][cw][lane] = mass;
                __syncwarp();
                if (lane == 0) mbar_arrive(&sh.s2_done[dslot]);
            }
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
