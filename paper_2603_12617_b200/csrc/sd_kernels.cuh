// The two kernels of the verify-and-feedback step.
//
//   sd_cluster_kernel  fast path.  One thread-block cluster per (sequence, row) unit; each block
//                      owns a contiguous slice of the vocabulary, pulls it into shared memory once
//                      with bulk asynchronous copies (cp.async.bulk + mbarrier), computes the
//                      softmax statistics from shared memory, exchanges them through distributed
//                      shared memory, and makes the second sweep (gradient, residual chunk sums)
//                      over the copy that is still resident.  HBM sees each logit once.
//   sd_generic_kernel  any V and any alignment.  One block per unit, two sweeps over global
//                      memory with element loads.  Same arithmetic, same workspace, same resolver.
//
// A unit is row i of sequence b: i < k pairs target row i with draft row i (Algorithm 1's
// rejection test, the KL loss of Eq. "kl_divergence" and its gradient); i == k is the bonus row.
// The block that takes the last ticket of a sequence resolves it (accept length, emitted tokens,
// inverse-CDF draw); nobody waits for anybody.
#pragma once

#include "sd_device.cuh"

namespace sdv {

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
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: false if the copy did not land within kWaitLimit polls.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < kWaitLimit; ++it)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// 1-D bulk copy global -> shared of this block, completion counted on `bar`.
// Both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes,
                                          uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
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

// Chunks [c0, c0+nc) of the row that block `rank` of `C` owns.
__device__ __forceinline__ void block_chunks(int NC, int C, int rank, int& c0, int& nc) {
    const int base = NC / C, rem = NC % C;
    nc = base + (rank < rem ? 1 : 0);
    c0 = rank * base + min(rank, rem);
}

struct ClusterShared {
    uint64_t bar[kMaxPieces];
    StatScratch stat;
    PartialStats xchg[kMaxCluster];   // written by every block of the cluster (distributed shared memory)
    RowConst rc;
    ResolveScratch rs;
};

// ---- fast path -----------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads) sd_cluster_kernel(const Params P, const int slice_chunks) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    constexpr int CE = kChunkVecs * VEC;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    __shared__ ClusterShared sh;

    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int unit = blockIdx.x / C;
    const int b = unit / (P.k + 1), i = unit % (P.k + 1);
    const bool bonus = (i == P.k);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int c0, nc;
    block_chunks(P.NC, C, rank, c0, nc);
    const int npieces = (nc + kPieceChunks - 1) / kPieceChunks;

    uint4* sT = reinterpret_cast<uint4*>(dyn_smem);
    uint4* sD = reinterpret_cast<uint4*>(dyn_smem + (size_t)slice_chunks * kChunkBytes);
    const typename E::type* Trow = reinterpret_cast<const typename E::type*>(P.T) + (size_t)unit * P.V;
    const typename E::type* Drow =
        reinterpret_cast<const typename E::type*>(P.D) + (size_t)(b * P.k + (bonus ? 0 : i)) * P.V;

    // -- issue every bulk copy of this block's slice up front
    if (tid == 0) {
        for (int p = 0; p < npieces; ++p) mbar_init(&sh.bar[p], 1);
        fence_barrier_init();
        fence_proxy_async();
        for (int p = 0; p < npieces; ++p) {
            const int q0 = p * kPieceChunks;
            const int nch = min(kPieceChunks, nc - q0);
            const int e0 = (c0 + q0) * CE;
            const int elems = min(nch * CE, P.V - e0);
            const uint32_t bytes = (uint32_t)elems * (uint32_t)sizeof(typename E::type);
            mbar_expect_tx(&sh.bar[p], bonus ? bytes : 2u * bytes);
            bulk_load(reinterpret_cast<unsigned char*>(sT) + (size_t)q0 * kChunkBytes, Trow + e0, bytes,
                      &sh.bar[p]);
            if (!bonus)
                bulk_load(reinterpret_cast<unsigned char*>(sD) + (size_t)q0 * kChunkBytes, Drow + e0, bytes,
                          &sh.bar[p]);
        }
    }
    // the thread that will report the row fetches what the accept test needs while the copies fly
    AcceptOperands aop;
    aop.valid = false;
    if (rank == 0 && tid == 0 && !bonus) aop = load_accept_operands<DT>(P, b, i);
    __syncthreads();          // barriers are initialised before anyone polls them
    cluster.barrier_arrive(); // matched by the wait before the first remote store: every block of
                              // the cluster must be running before its shared memory is written

    // -- sweep 1 (shared memory): online softmax statistics, one reference per lane
    LaneStats ls;
    ls.init(P.c);
    bool timed_out = false;
    for (int q = warp; q < nc; q += kWarps) {
        if (!mbar_wait_bounded(&sh.bar[q / kPieceChunks], 0)) { timed_out = true; break; }
        const int ebase = (c0 + q) * CE;
#pragma unroll
        for (int j = 0; j < kChunkVecs / 32; ++j) {
            const int vi = j * 32 + lane;
            if (ebase + vi * VEC < P.V) {
                float t[VEC];
                E::unpack(sT[q * kChunkVecs + vi], t);
                if (!bonus) {
                    float d[VEC];
                    E::unpack(sD[q * kChunkVecs + vi], d);
                    ls.template add_pair<VEC>(t, d, P.c);
                } else {
                    ls.template add_bonus<VEC>(t, P.c);
                }
            }
        }
    }
    if (timed_out && lane == 0) atomicOr(&P.wstatus[b], kStatusTimeout);
    const PartialStats mine = block_reduce_stats(ls, P.c, sh.stat);   // same in every thread

    // -- block statistics to every block of the cluster
    cluster.barrier_wait();
    if (warp == 0 && lane < C) *cluster.map_shared_rank(&sh.xchg[rank], lane) = mine;
    cluster.sync();   // all partials of the row are now in this block's shared memory

    if (warp == 0) {
        const PartialStats row = warp_merge_partials(sh.xchg, C, P.c);
        const RowConst rcw = row_constants(P, bonus, row);
        if (lane == 0) sh.rc = rcw;
        __syncwarp();
        // one thread of the cluster reports the row: loss, accept flag, constants for the resolver
        if (rank == 0 && lane == 0) finish_row(P, b, i, row, rcw, aop);
    }
    __syncthreads();
    const RowConst rc = sh.rc;

    // -- sweep 2 (shared memory): gradient out, residual / bonus mass per sampling chunk
    typename E::type* Grow =
        P.grad ? reinterpret_cast<typename E::type*>(P.grad) + (size_t)(b * P.k + (bonus ? 0 : i)) * P.V
               : nullptr;
    float* csum = P.chunk_sums + (size_t)unit * P.NC;
    for (int q = warp; q < nc; q += kWarps) {
        const int ebase = (c0 + q) * CE;
        float mass = 0.f;
#pragma unroll
        for (int j = 0; j < kChunkVecs / 32; ++j) {
            const int vi = j * 32 + lane;
            const int e = ebase + vi * VEC;
            if (e < P.V) {
                float t[VEC];
                E::unpack(sT[q * kChunkVecs + vi], t);
                if (!bonus) {
                    float d[VEC], g[VEC];
                    E::unpack(sD[q * kChunkVecs + vi], d);
#pragma unroll
                    for (int z = 0; z < VEC; ++z) {
                        g[z] = grad_elem(t[z], d[z], P.c, rc);
                        mass += fmaxf(-g[z], 0.f);
                    }
                    if (Grow) store_streaming(Grow + e, E::pack(g));
                } else {
#pragma unroll
                    for (int z = 0; z < VEC; ++z) mass += prob_elem(t[z], P.c, rc);
                }
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) mass += __shfl_xor_sync(0xffffffffu, mass, off);
        if (lane == 0) csum[c0 + q] = mass;
    }

    // -- last block of the sequence resolves it
    if (take_ticket(P, b, &sh.rs.ticket_last)) resolve_sequence<DT>(P, b, sh.rs);
}

// ---- generic path --------------------------------------------------------------------------
struct GenericShared {
    StatScratch stat;
    RowConst rc;
    ResolveScratch rs;
};

template <int DT>
__global__ void __launch_bounds__(kThreads) sd_generic_kernel(const Params P) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    constexpr int CE = kChunkVecs * VEC;
    __shared__ GenericShared sh;

    const int unit = blockIdx.x;
    const int b = unit / (P.k + 1), i = unit % (P.k + 1);
    const bool bonus = (i == P.k);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t offT = (size_t)unit * P.V;
    const size_t offD = (size_t)(b * P.k + (bonus ? 0 : i)) * P.V;

    // sweep 1: statistics; lanes take consecutive elements
    LaneStats ls;
    ls.init(P.c);
    for (int q = warp; q < P.NC; q += kWarps) {
        const int ebase = q * CE;
        for (int j = lane; j < CE; j += 32) {
            const int v = ebase + j;
            if (v < P.V) {
                float t[1] = {E::load(P.T, offT + v)};
                if (!bonus) {
                    float d[1] = {E::load(P.D, offD + v)};
                    ls.template add_pair<1>(t, d, P.c);
                } else {
                    ls.template add_bonus<1>(t, P.c);
                }
            }
        }
    }
    {
        const PartialStats row = block_reduce_stats(ls, P.c, sh.stat);
        if (tid == 0) {
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

    // sweep 2: gradient and chunk sums
    float* csum = P.chunk_sums + (size_t)unit * P.NC;
    for (int q = warp; q < P.NC; q += kWarps) {
        const int ebase = q * CE;
        float mass = 0.f;
        for (int j = lane; j < CE; j += 32) {
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
        if (lane == 0) csum[q] = mass;
    }

    if (take_ticket(P, b, &sh.rs.ticket_last)) resolve_sequence<DT>(P, b, sh.rs);
}

}  // namespace sdv
