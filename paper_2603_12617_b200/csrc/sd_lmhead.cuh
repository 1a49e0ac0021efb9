// The step after the feedback: the gradient of the round's loss with respect to the weights of the
// draft model's (linear) output layer,
//     dW[v,j] = sum_r g[r,v] * x[r,j]          dW = g^T X,   g [R,V] (gradient w.r.t. the draft logits,
//                                               Sec. 3.1), X [R,d] (hidden states), R = B*k positions,
// a dense contraction over the positions of the round: the one place on this path where the
// tensor cores apply.  sm_100a: operands by TMA (cp.async.bulk.tensor) into 128-byte-swizzled
// shared memory, tcgen05.mma (bf16 x bf16 -> fp32) with the accumulator in tensor memory,
// tcgen05.ld for the epilogue.
//
// Both operands have the contracted index r as their slow index in memory, so both are "MN-major"
// operands of the instruction: a tile of g is [64 positions][128 vocabulary entries] with the
// vocabulary entries contiguous, a tile of X is [64 positions][256 features] likewise.
//
// One block per SM, persistent over output tiles of 128 x 256; the features run fastest over the
// tiles, so the blocks that work at the same time share a few tiles of g (each read from HBM once)
// and all of X (which stays in L2).  Warp roles:
//   warp 0      producer: one thread issues the TMA loads of a stage (6 boxes of 64 x 64 bf16)
//   warp 1      one thread issues the MMAs (4 of K = 16 per stage) and the commits
//   warps 2..5  epilogue: tensor memory -> registers -> a staging block in shared memory -> global
//               memory in whole 128-byte lines, while the MMAs of the next tile fill the other half
//               of tensor memory.  (A lane gets 32 consecutive columns of ONE row from tensor memory;
//               stored from there, every instruction of a warp touches 32 different lines with 16
//               bytes each, and the result -- 2.1 GB at the full size -- left at 1.4 TB/s.)
// Every wait is bounded; a wait that gives up sets an error word, and the block frees its tensor
// memory and returns.  No multicast, no cluster.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sd_kernels.cuh"

namespace sdv {

constexpr int kGemmBM = 128;                 // vocabulary entries per tile (rows of dW)
constexpr int kGemmBN = 256;                 // features per tile (columns of dW)
constexpr int kGemmBK = 64;                  // positions per stage
constexpr int kGemmStages = 4;
constexpr int kGemmChunk = 64;               // entries of a 128-byte swizzled row (bf16)
constexpr int kGemmChunkBytes = kGemmBK * kGemmChunk * 2;            // one TMA box: 8 KiB
constexpr int kGemmABytes = (kGemmBM / kGemmChunk) * kGemmChunkBytes;   // 16 KiB
constexpr int kGemmBBytes = (kGemmBN / kGemmChunk) * kGemmChunkBytes;   // 32 KiB
constexpr int kGemmStageBytes = kGemmABytes + kGemmBBytes;            // 48 KiB
constexpr int kGemmThreads = 6 * 32;
constexpr int kGemmTmemCols = 512;           // two accumulators of 128 lanes x 256 fp32 columns
constexpr int kGemmStagingStride = 36;       // floats per staged row: 32 + 4, keeps 16-byte accesses conflict-free
constexpr int kGemmStagingBytes = 32 * kGemmStagingStride * 4;   // per epilogue warp
constexpr int kGemmSmem = kGemmStages * kGemmStageBytes + 4 * kGemmStagingBytes + 1024 /* alignment */ + 256 /* barriers */;
constexpr long long kGemmWaitCycles = 4000000000ll;   // about two seconds

struct GemmParams {
    int R, V, d;
    float* out;              // [V,d]
    uint32_t* error;         // set when a bounded wait gave up
};

// ---- PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_2d(void* dst_smem, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
            smem_u32(dst_smem)),
        "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot_in_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_in_smem)), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// D[tmem] (+)= A[smem] * B[smem]; accumulate = 0 overwrites D.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier gets one arrival when every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory: thread i of the warp gets lane i.
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]),
          "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]),
          "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor of an MN-major tile in the 128-byte swizzle: rows of 64 bf16
// along M (or N), 128 bytes apart along K, eight of them to a swizzle atom.  lbo: bytes from one
// group of 64 entries along M/N to the next; sbo: bytes from one group of 8 positions along K to
// the next.  (Bits 0-13 address >> 4, 16-29 lbo >> 4, 32-45 sbo >> 4, 46-47 version 1, 61-63 swizzle 128 B = 2.)
__device__ __forceinline__ uint64_t umma_desc_mn_sw128(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands MN-major, M x N.
__host__ __device__ constexpr uint32_t umma_idesc_bf16_mn(int M, int N) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// Bounded wait on a barrier of this block by one thread; false (and the error word set) when it gives up.
__device__ __forceinline__ bool gemm_wait(uint64_t* bar, uint32_t parity, volatile int* abort, uint32_t* error) {
    long long t0 = 0;
    for (uint32_t it = 0;; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 255u) == 255u) {
            if (*abort) return false;
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > kGemmWaitCycles) break;
        }
    }
    *abort = 1;
    atomicExch(error, 1u);
    return false;
}

struct GemmShared {
    uint64_t full[kGemmStages];      // stage filled by TMA                 (1 arrival + bytes)
    uint64_t empty[kGemmStages];     // stage read by the MMAs              (1: commit)
    uint64_t acc_full[2];            // accumulator complete                (1: commit)
    uint64_t acc_empty[2];           // accumulator read by the epilogue    (4: one per epilogue warp)
    uint32_t tmem_base;
    int abort;
};

__global__ void __launch_bounds__(kGemmThreads, 1)
sd_lmhead_kernel(const __grid_constant__ CUtensorMap map_g, const __grid_constant__ CUtensorMap map_x, const GemmParams P) {
    extern __shared__ unsigned char gemm_smem_raw[];
    unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(gemm_smem_raw) + 1023) & ~(uintptr_t)1023);
    float* staging_all = reinterpret_cast<float*>(smem + kGemmStages * kGemmStageBytes);
    GemmShared& sh = *reinterpret_cast<GemmShared*>(smem + kGemmStages * kGemmStageBytes + 4 * kGemmStagingBytes);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    volatile int* abort = &sh.abort;

    const int tiles_m = (P.V + kGemmBM - 1) / kGemmBM, tiles_n = (P.d + kGemmBN - 1) / kGemmBN;
    const long long tiles = (long long)tiles_m * tiles_n;
    const int kblocks = (P.R + kGemmBK - 1) / kGemmBK;

    if (tid == 0) {
        for (int s = 0; s < kGemmStages; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&sh.acc_full[a], 1); mbar_init(&sh.acc_empty[a], 4); }
        sh.abort = 0;
        fence_barrier_init();
        fence_proxy_async();
    }
    if (warp == 1) tmem_alloc(&sh.tmem_base, kGemmTmemCols);     // the whole warp; the same warp frees it
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;

    if (warp == 0) {
        // ---- producer
        if (lane == 0) {
            int stage = 0;
            uint32_t par = 1;                  // parity of the stage's previous use on empty[]
            long long n = 0;                   // stages issued so far
            bool ok = true;
            for (long long tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int m0 = (int)(tile / tiles_n) * kGemmBM, n0 = (int)(tile % tiles_n) * kGemmBN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (n >= kGemmStages && !gemm_wait(&sh.empty[stage], par, abort, P.error)) { ok = false; break; }
                    unsigned char* a = smem + (size_t)stage * kGemmStageBytes;
                    unsigned char* b = a + kGemmABytes;
                    mbar_expect_tx(&sh.full[stage], (uint32_t)kGemmStageBytes);   // boxes out of range still count in full
                    const int r0 = kb * kGemmBK;
#pragma unroll
                    for (int c = 0; c < kGemmBM / kGemmChunk; ++c)
                        tma_load_2d(a + c * kGemmChunkBytes, &map_g, m0 + c * kGemmChunk, r0, &sh.full[stage]);
#pragma unroll
                    for (int c = 0; c < kGemmBN / kGemmChunk; ++c)
                        tma_load_2d(b + c * kGemmChunkBytes, &map_x, n0 + c * kGemmChunk, r0, &sh.full[stage]);
                    ++n;
                    if (++stage == kGemmStages) { stage = 0; par ^= 1u; }
                }
            }
            // leaving early: every load issued has landed before the block goes away
            if (!ok) {
                const long long t0 = clock64();
                for (long long i = (n > kGemmStages ? n - kGemmStages : 0); i < n; ++i) {
                    const uint32_t p = (uint32_t)(i / kGemmStages) & 1u;
                    while (!mbar_try_wait(&sh.full[i % kGemmStages], p))
                        if (clock64() - t0 > kGemmWaitCycles) break;
                }
            }
        }
    } else if (warp == 1) {
        // ---- MMA issuer
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16_mn(kGemmBM, kGemmBN);
            int stage = 0;
            uint32_t par = 0;
            long long it = 0;                  // tiles of this block so far
            bool ok = true;
            for (long long tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++it) {
                const int acc = (int)(it & 1);
                // the epilogue must have read this accumulator's previous tile
                if (it >= 2 && !gemm_wait(&sh.acc_empty[acc], (uint32_t)((it >> 1) - 1) & 1u, abort, P.error)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem + (uint32_t)acc * kGemmBN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    if (!gemm_wait(&sh.full[stage], par, abort, P.error)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t a = smem_u32(smem + (size_t)stage * kGemmStageBytes);
                    const uint32_t b = a + kGemmABytes;
#pragma unroll
                    for (int k4 = 0; k4 < kGemmBK / 16; ++k4) {
                        // 16 positions further: 16 rows of 128 bytes
                        const uint64_t da = umma_desc_mn_sw128(a + k4 * 16 * 128, kGemmChunkBytes, 1024);
                        const uint64_t db = umma_desc_mn_sw128(b + k4 * 16 * 128, kGemmChunkBytes, 1024);
                        umma_bf16(d_tmem, da, db, idesc, (kb | k4) != 0 ? 1u : 0u);
                    }
                    umma_commit(&sh.empty[stage]);          // the stage is free once these MMAs have read it
                    if (++stage == kGemmStages) { stage = 0; par ^= 1u; }
                }
                if (ok) umma_commit(&sh.acc_full[acc]);
            }
        }
    } else {
        // ---- epilogue: warp w reads the tensor-memory lanes 32*(w%4) .. +31 (rows of the tile)
        const int q = warp & 3;
        long long it = 0;
        bool ok = true;
        for (long long tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++it) {
            const int acc = (int)(it & 1);
            const int m0 = (int)(tile / tiles_n) * kGemmBM, n0 = (int)(tile % tiles_n) * kGemmBN;
            int got = 1;
            if (lane == 0) got = gemm_wait(&sh.acc_full[acc], (uint32_t)(it >> 1) & 1u, abort, P.error) ? 1 : 0;
            got = __shfl_sync(0xffffffffu, got, 0);
            if (!got) { ok = false; break; }
            tc_fence_after();
            float* stg = staging_all + (size_t)(warp - 2) * (kGemmStagingBytes / 4);
            const int vbase = m0 + q * 32;               // first row of this warp's 32
#pragma unroll 1
            for (int c = 0; c < kGemmBN / 32; ++c) {
                uint32_t r[32];
                tmem_ld_32x32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kGemmBN + c * 32), r);
                tmem_ld_wait();
                // lane = row of the block: 32 columns into the staging block
#pragma unroll
                for (int e = 0; e < 32; e += 4)
                    *reinterpret_cast<float4*>(stg + lane * kGemmStagingStride + e) =
                        make_float4(__uint_as_float(r[e]), __uint_as_float(r[e + 1]), __uint_as_float(r[e + 2]),
                                    __uint_as_float(r[e + 3]));
                __syncwarp();
                // eight lanes per row now: every store instruction writes four whole 128-byte lines
                const int j0 = n0 + c * 32;
                const int cr = lane >> 3, cc = (lane & 7) * 4;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = i * 4 + cr;
                    const int v = vbase + rr;
                    const float4 val = *reinterpret_cast<const float4*>(stg + rr * kGemmStagingStride + cc);
                    if (v < P.V) {
                        float* dst = P.out + (size_t)v * P.d + j0 + cc;
                        if (j0 + cc + 4 <= P.d) {
                            __stcs(reinterpret_cast<float4*>(dst), val);
                        } else {
                            const float t4[4] = {val.x, val.y, val.z, val.w};
                            for (int e = 0; e < 4; ++e)
                                if (j0 + cc + e < P.d) dst[e] = t4[e];
                        }
                    }
                }
                __syncwarp();
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.acc_empty[acc]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem, kGemmTmemCols);
}

}  // namespace sdv
