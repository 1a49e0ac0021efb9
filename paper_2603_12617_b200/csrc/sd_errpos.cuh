// Error-position feedback (the feedback OSD collects, Sec. 3.1 "Online Update with Gradient
// Descent": the positions where the draft was wrong, with the target's logits there).  Per sequence
// only the first rejected position n_b feeds the update: its gradient row is all that is written,
// and it is also the only row whose masses the residual draw needs (the bonus row when every draft
// token was accepted).  So the step splits in two kernels:
//
//   sd_stream_kernel<DT, false, STATS>   pass 1 of every row: row constants, losses, rejection tests
//   sd_errpos_kernel                     this file: for each sequence the one row it still needs --
//                                        gradient of row n_b (same instructions as pass 2 of the
//                                        full step), the masses of its sampling regions, and the
//                                        draw by the block that takes the sequence's last ticket.
//
// The row is read straight from global memory (2 x kRegionRows 16-byte loads in flight per lane); a block
// takes a slice of kErrSliceRegions sampling regions, a warp one region at a time.
#pragma once

#include "sd_kernels.cuh"

namespace sdv {

constexpr int kErrThreads = 256;
constexpr int kErrSliceRegions = 32;

template <int DT>
__global__ void __launch_bounds__(kErrThreads, 4) sd_errpos_kernel(const __grid_constant__ Params P, const int slices) {
    using E = Elem<DT>;
    using ET = typename E::type;
    constexpr int VEC = E::VEC;
    constexpr int kGroups = kRegionRows;            // a region is kRegionRows x 32 vectors, as in the streaming kernel
    __shared__ int is_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = (int)blockIdx.x / slices, sl = (int)blockIdx.x - b * slices;
    const int k = P.k;

    // first rejected position (flags written by the kernel before this one)
    int n = k;
    for (int i = 0; i < k; ++i)
        if (P.accept[b * k + i] == 0) { n = i; break; }
    const bool bonus = (n == k);
    const int unit = b * (k + 1) + n;
    const RowConst rc = P.rowc[unit];
    const uint4* Trow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.T) + (size_t)unit * P.V);
    const uint4* Drow = reinterpret_cast<const uint4*>(reinterpret_cast<const ET*>(P.D) + (size_t)(b * k + (bonus ? 0 : n)) * P.V);
    uint4* Grow = P.grad ? reinterpret_cast<uint4*>(reinterpret_cast<ET*>(P.grad) + (size_t)b * P.V) : nullptr;
    const int NV = P.V / VEC;
    const int RV = P.RE / VEC;                      // vectors per region: kGroups * 32
    float* rsum = P.region_sums + (size_t)unit * P.NR;
    const int r0 = sl * kErrSliceRegions, r1 = min(P.NR, r0 + kErrSliceRegions);

    for (int r = r0 + warp; r < r1; r += kErrThreads / 32) {
        const int v0 = r * RV;
        const int nv = min(RV, NV - v0);
        if (!SD_IN(r, P.NR, 50) || !SD_IN((long long)(v0 + nv) * VEC - 1, P.V, 51) || !SD_IN(unit, P.B * (k + 1), 52)) continue;
        uint4 rt[kGroups], rd[kGroups];
#pragma unroll
        for (int g = 0; g < kGroups; ++g) {
            const int vi = g * 32 + lane;
            rt[g] = vi < nv ? __ldcs(Trow + v0 + vi) : E::masked();
            rd[g] = (!bonus && vi < nv) ? __ldcs(Drow + v0 + vi) : E::masked();
        }
        // the arithmetic of pass 2 of the full step, instruction for instruction
        float mass;
        if (!bonus) {
            mass = pass2_region<DT, false>(rt, rd, nv, lane, P.c, rc,
                                           Grow ? reinterpret_cast<ET*>(Grow + v0) : nullptr);
        } else {
            mass = pass2_region<DT, true>(rt, rd, nv, lane, P.c, rc, nullptr);
            if (Grow) {
#pragma unroll
                for (int g = 0; g < kGroups; ++g) {
                    const int vi = g * 32 + lane;
                    if (vi < nv) __stcs(Grow + v0 + vi, make_uint4(0u, 0u, 0u, 0u));   // no error position: a zero row
                }
            }
        }
        if (lane == 0) rsum[r] = mass;
    }

    // the block's masses are out before its ticket is; the last ticket of the sequence draws
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const uint32_t old = atomicAdd(P.ticket + b, 1u);
        is_last = (old == (uint32_t)slices - 1u);
        if (is_last) __threadfence();
    }
    __syncthreads();
    if (is_last && warp == 0) resolve_sequence<DT, true>(P, b);   // also sets ticket and status words back to zero
}

}  // namespace sdv
