// Sub-bit budgets (EDEN Section 4.1): the shared-seed sparsification mask with exactly k
// ones, its application before the rotation (gather + 1/p rescale, the factor being
// folded into the scale S) and its inverse on the receiver (scatter into the sum).
//
// The mask keeps the k coordinates with the smallest (key, index) pairs, key_i being the
// 32-bit Philox stream-1 word of coordinate i.  The k-th smallest pair is found exactly
// with two 16-bit histogram rounds; a coordinate is then kept iff key < tau, or key ==
// tau and fewer than `rem` equal keys precede it.  Positions in the compacted vector are
// exclusive prefix counts: per 1024-coordinate chunk counts, a scan of the chunk counts,
// and a block scan inside each chunk.
#pragma once
#include "eden_device.cuh"

namespace eden {

constexpr int kSelThreads = 256;
constexpr int kSelChunk = kSelThreads * 4;   // coordinates per block in the chunk kernels

// Histogram of key bits: round 0 counts the top 16 bits of every key; round 1 counts the
// low 16 bits of the keys whose top bits equal sel->bin_hi.
__global__ void __launch_bounds__(kSelThreads)
k_sel_hist(uint64_t seed, uint64_t d, int round, const MaskSelect* __restrict__ sel,
           uint32_t* __restrict__ hist)
{
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t * 4 >= d) return;
    const uint4 k4 = mask_keys(seed, t);
    const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
    const uint32_t want = round ? sel->bin_hi : 0u;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        if (t * 4 + j >= d) break;
        if (round == 0) atomicAdd(&hist[keys[j] >> 16], 1u);
        else if ((keys[j] >> 16) == want) atomicAdd(&hist[keys[j] & 0xFFFFu], 1u);
    }
}

// Finds the histogram bin that holds the element of 0-based rank r (one block of 1024
// threads over 65536 bins).  Round 0: r = k - 1, writes bin_hi / below_hi.  Round 1:
// r = k - 1 - below_hi, writes tau, below and rem.
__global__ void __launch_bounds__(1024)
k_sel_find(const uint32_t* __restrict__ hist, uint64_t k, int round, MaskSelect* __restrict__ sel)
{
    __shared__ unsigned long long scratch[33];
    const uint32_t r = round ? (uint32_t)(k - 1) - sel->below_hi : (uint32_t)(k - 1);
    uint32_t mine = 0;
    for (int j = 0; j < 64; ++j) mine += hist[threadIdx.x * 64 + j];
    unsigned long long total;
    const uint32_t before = (uint32_t)block_exclusive_scan(mine, scratch, &total);
    if (r >= before && r < before + mine) {
        uint32_t run = before;
        for (int j = 0; j < 64; ++j) {
            const uint32_t h = hist[threadIdx.x * 64 + j];
            if (r < run + h) {
                const uint32_t bin = threadIdx.x * 64 + j;
                if (round == 0) {
                    sel->bin_hi = bin;
                    sel->below_hi = run;
                } else {
                    sel->tau = (sel->bin_hi << 16) | bin;
                    sel->below = sel->below_hi + run;
                    sel->rem = (uint32_t)k - (sel->below_hi + run);   // ties to keep, >= 1
                }
                break;
            }
            run += h;
        }
    }
}

// (keys below tau, keys equal to tau) of the four coordinates of Philox call t, as a
// packed pair: low 32 bits = below, high 32 bits = equal.
__device__ __forceinline__ unsigned long long classify4(uint64_t seed, uint64_t t, uint64_t d,
                                                        uint32_t tau, uint32_t cls[4])
{
    const uint4 k4 = mask_keys(seed, t);
    const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
    unsigned long long packed = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        cls[j] = 0;
        if (t * 4 + j < d) {
            if (keys[j] < tau) { cls[j] = 1; packed += 1ull; }
            else if (keys[j] == tau) { cls[j] = 2; packed += 1ull << 32; }
        }
    }
    return packed;
}

// Per chunk of 1024 coordinates: how many keys are below tau and how many equal it.
__global__ void __launch_bounds__(kSelThreads)
k_sel_chunk_count(uint64_t seed, uint64_t d, const MaskSelect* __restrict__ sel,
                  unsigned long long* __restrict__ chunk_counts)
{
    __shared__ unsigned long long scratch[33];
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t cls[4];
    const unsigned long long mine = classify4(seed, t, d, sel->tau, cls);
    unsigned long long total;
    block_exclusive_scan(mine, scratch, &total);
    if (threadIdx.x == 0) chunk_counts[blockIdx.x] = total;
}

// Exclusive scan of the packed chunk counts, in place (one block).
__global__ void __launch_bounds__(1024)
k_sel_chunk_scan(unsigned long long* __restrict__ chunk_counts, uint64_t n_chunks)
{
    __shared__ unsigned long long scratch[33];
    const uint64_t per = (n_chunks + blockDim.x - 1) / blockDim.x;
    const uint64_t lo = threadIdx.x * per, hi = min(lo + per, n_chunks);
    unsigned long long mine = 0;
    for (uint64_t j = lo; j < hi; ++j) mine += chunk_counts[j];
    unsigned long long total;
    unsigned long long run = block_exclusive_scan(mine, scratch, &total);
    for (uint64_t j = lo; j < hi; ++j) {
        const unsigned long long v = chunk_counts[j];
        chunk_counts[j] = run;
        run += v;
    }
}

enum SelectAction { SEL_COMPACT = 0, SEL_SCATTER_ACC = 1, SEL_MASK_BITS = 2 };

// Walks the coordinates in order, knowing for each whether it is kept and its position
// among the kept ones.
//   SEL_COMPACT:      y[pos] = x[i]                  (sender; the 1/p factor goes into S)
//   SEL_SCATTER_ACC:  out[i] += yhat[pos]            (receiver; Section 4.1: the receiver
//                                                     restores through the same mask)
//   SEL_MASK_BITS:    bit i of the bitmap = kept
template <int ACTION>
__global__ void __launch_bounds__(kSelThreads)
k_sel_apply(uint64_t seed, uint64_t d, const MaskSelect* __restrict__ sel,
            const unsigned long long* __restrict__ chunk_offsets,
            const float* __restrict__ in, float* __restrict__ out, uint32_t* __restrict__ bits)
{
    __shared__ unsigned long long scratch[33];
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t tau = sel->tau, rem = sel->rem;
    uint32_t cls[4];
    const unsigned long long mine = classify4(seed, t, d, tau, cls);
    unsigned long long total;
    const unsigned long long before = block_exclusive_scan(mine, scratch, &total) + chunk_offsets[blockIdx.x];
    uint32_t below = (uint32_t)before, ties = (uint32_t)(before >> 32);
    uint32_t nibble = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t i = t * 4 + j;
        bool keep = false;
        if (cls[j] == 1) keep = true;
        else if (cls[j] == 2) keep = ties < rem;
        if (keep) {
            const uint64_t pos = (uint64_t)below + min(ties, rem);
            if (ACTION == SEL_COMPACT) out[pos] = in[i];
            if (ACTION == SEL_SCATTER_ACC) out[i] += in[pos];
            nibble |= 1u << j;
        }
        if (cls[j] == 1) ++below;
        if (cls[j] == 2) ++ties;
    }
    if (ACTION == SEL_MASK_BITS) {
        uint32_t w = nibble << (4 * (threadIdx.x & 7));
        w |= __shfl_xor_sync(0xffffffffu, w, 1);
        w |= __shfl_xor_sync(0xffffffffu, w, 2);
        w |= __shfl_xor_sync(0xffffffffu, w, 4);
        if ((threadIdx.x & 7) == 0 && t * 4 < d) bits[t >> 3] = w;
    }
}

}  // namespace eden
