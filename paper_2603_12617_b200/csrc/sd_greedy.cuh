// Greedy verification (Algorithm 1 in the limit tau -> 0; the decoding mode of the paper's
// experiments, Sec. 4.1): a draft token is accepted iff it is the target's argmax of its position,
// and the extra token is the target's argmax at the first mismatch (or at the bonus position).
// Only the target logits are read, once: the kernel is a streaming argmax, bound by HBM.
//
//   sd_greedy_kernel   grid-stride over items (a row cut into pieces of kGreedyItemVecs 16-byte
//                      vectors).  Every thread keeps the largest value it has seen and its first
//                      index, a warp folds them into one 64-bit key (value in an order-preserving
//                      integer form, then the complement of the index, so that the larger key is the
//                      larger value and, among equals, the smaller index) and applies it to the row's
//                      key with one atomicMax whose result nobody reads.  Warps never wait for one
//                      another inside the loop.  A block that has run out of items takes a ticket;
//                      the block with the last ticket reads all keys, compares them with the draft
//                      tokens and writes accept lengths and tokens.  Nobody waits for anybody.
#pragma once

#include "sd_device.cuh"

namespace sdv {

constexpr int kGreedyThreads = 256;
constexpr int kGreedyItemVecs = 8 * kGreedyThreads;   // 32 KiB of a row per item: 8 loads in flight per thread

struct GreedyParams {
    const void* T;            // [B,k+1,V]
    const int32_t* x;         // [B,k]
    int B, k, V;
    int items_per_row;
    int vectorised;           // rows start on 16-byte boundaries and hold whole vectors
    int32_t* accept_len;      // [B]
    int32_t* tokens;          // [B,k+1]
    int32_t* argmax;          // [B,k+1] or null
    unsigned long long* keys; // [B*(k+1)] zero on entry and zero again on exit
    uint32_t* ticket;         // one word, zero on entry and zero again on exit
};

// Larger value -> larger key; equal values -> smaller index -> larger key.  v is not NaN.
__device__ __forceinline__ unsigned long long greedy_key(float v, int idx) {
    const uint32_t u = __float_as_uint(v + 0.f);                 // -0 becomes +0: equal values, equal keys
    const uint32_t ord = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ((unsigned long long)ord << 32) | (uint32_t)(0x7fffffff - idx);
}
__device__ __forceinline__ int greedy_index(unsigned long long key) {
    return key == 0ull ? 0 : 0x7fffffff - (int)(uint32_t)(key & 0xffffffffu);   // untouched key: a row without a finite or +inf entry
}

template <int DT>
__global__ void __launch_bounds__(kGreedyThreads) sd_greedy_kernel(const GreedyParams P) {
    using E = Elem<DT>;
    constexpr int VEC = E::VEC;
    __shared__ int is_last;
    const int tid = threadIdx.x, lane = tid & 31;
    const int K1 = P.k + 1;
    const long long items = (long long)P.B * K1 * P.items_per_row;
    const int item_elems = kGreedyItemVecs * VEC;

    for (long long it = blockIdx.x; it < items; it += gridDim.x) {
        const int row = (int)(it / P.items_per_row);
        const int piece = (int)(it - (long long)row * P.items_per_row);
        const int e0 = piece * item_elems;
        const int n = min(item_elems, P.V - e0);           // entries of this item
        if (!SD_IN(row, (long long)P.B * K1, 40) || !SD_IN(e0 + n - 1, P.V, 41)) continue;
        float best = -INFINITY;
        int besti = 0x7fffffff;
        if (P.vectorised) {
            const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const typename E::type*>(P.T) +
                                                              (size_t)row * P.V + e0);
            const int nvec = n / VEC;
            uint4 q[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int vi = j * kGreedyThreads + tid;
                q[j] = vi < nvec ? __ldcs(src + vi) : E::masked();
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int vi = j * kGreedyThreads + tid;
                float v[VEC];
                E::unpack(q[j], v);
#pragma unroll
                for (int e = 0; e < VEC; ++e)
                    if (v[e] > best) { best = v[e]; besti = e0 + vi * VEC + e; }   // strict: keeps the first index
            }
        } else {
            for (int j = tid; j < n; j += kGreedyThreads) {
                const float v = E::load(P.T, (size_t)row * P.V + e0 + j);
                if (v > best) { best = v; besti = e0 + j; }
            }
        }
        unsigned long long key = best > -INFINITY ? greedy_key(best, besti) : 0ull;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const unsigned long long o = __shfl_xor_sync(0xffffffffu, key, off);
            key = o > key ? o : key;
        }
        if (lane == 0 && key != 0ull) atomicMax(P.keys + row, key);
    }

    // this block's keys are out before its ticket is
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const uint32_t old = atomicAdd(P.ticket, 1u);
        is_last = (old == gridDim.x - 1);
        if (is_last) __threadfence();
    }
    __syncthreads();
    if (!is_last) return;

    // every key is final: accept length and tokens, one thread per sequence; the keys go back to
    // zero on the way, so that the scratch is ready for the next call
    for (int b = tid; b < P.B; b += kGreedyThreads) {
        unsigned long long* kb = P.keys + (size_t)b * K1;
        const int32_t* xb = P.x + (size_t)b * P.k;
        int32_t* tb = P.tokens + (size_t)b * K1;
        int n_acc = -1, y = 0;
        for (int i = 0; i <= P.k; ++i) {
            const int am = greedy_index(__ldcg(kb + i));
            kb[i] = 0ull;
            if (P.argmax) P.argmax[(size_t)b * K1 + i] = am;
            if (n_acc < 0 && (i == P.k || xb[i] != am)) { n_acc = i; y = am; }
            tb[i] = (n_acc < 0) ? am : (i == n_acc ? y : -1);   // accepted draft token = the argmax
        }
        P.accept_len[b] = n_acc;
    }
    if (tid == 0) *P.ticket = 0;   // leave the word ready for the next call
}

}  // namespace sdv
