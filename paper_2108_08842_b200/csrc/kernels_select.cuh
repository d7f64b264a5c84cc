// Sub-bit budgets (EDEN Section 4.1): the shared-seed sparsification mask with exactly k
// ones, its application before the rotation (gather + 1/p rescale, the factor being
// folded into the scale S) and its inverse on the receiver (scatter into the sum).
//
// The mask keeps the k coordinates with the smallest (key, index) pairs, key_i being the
// 32-bit Philox stream-1 word of coordinate i.  The k-th smallest pair is found exactly:
// a coordinate is kept iff key < tau, or key == tau and fewer than `rem` equal keys
// precede it.  Positions in the compacted vector are exclusive prefix counts: per
// 1024-coordinate chunk counts, a scan of the chunk counts, and a scan inside each chunk.
// Three forms: single-job kernels with two 16-bit histogram rounds (the mask entry points),
// batched kernels with three digit rounds over all keys (long vectors), and the batched
// form with a candidate list and a mask bitmap (the default), which reads the keys once
// where the threshold falls inside the band predicted for it and twice otherwise.
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
// r = k - 1 - below_hi, writes tau, below and rem.  Each warp sums a run of 2048 bins with
// coalesced loads; the warp whose run holds rank r then walks it 32 bins at a time.
__device__ __forceinline__ void sel_find_body(const uint32_t* __restrict__ hist, uint64_t k, int round,
                                              MaskSelect* __restrict__ sel)
{
    __shared__ uint32_t warp_total[32];
    __shared__ uint32_t warp_before[32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t r = round ? (uint32_t)(k - 1) - sel->below_hi : (uint32_t)(k - 1);
    const uint32_t* run = hist + warp * 2048;
    uint32_t mine = 0;
#pragma unroll 8
    for (int i = 0; i < 64; ++i) mine += run[i * 32 + lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if (lane == 0) warp_total[warp] = mine;
    __syncthreads();
    if (warp == 0) {
        const uint32_t v = warp_total[lane];
        uint32_t inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        warp_before[lane] = inc - v;
    }
    __syncthreads();
    const uint32_t before = warp_before[warp];
    if (r >= before && r < before + warp_total[warp]) {        // exactly one warp
        uint32_t seen = before;
        for (int i = 0; i < 64; ++i) {
            const uint32_t v = run[i * 32 + lane];
            uint32_t inc = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += t;
            }
            const uint32_t chunk_total = __shfl_sync(0xffffffffu, inc, 31);
            if (r < seen + chunk_total) {
                const uint32_t hit = __ballot_sync(0xffffffffu, r < seen + inc);
                const int first = __ffs(hit) - 1;
                if (lane == first) {
                    const uint32_t bin = (uint32_t)(warp * 2048 + i * 32 + lane);
                    const uint32_t below = seen + inc - v;
                    if (round == 0) {
                        sel->bin_hi = bin;
                        sel->below_hi = below;
                    } else {
                        sel->tau = (sel->bin_hi << 16) | bin;
                        sel->below = sel->below_hi + below;
                        sel->rem = (uint32_t)k - (sel->below_hi + below);   // ties to keep, >= 1
                    }
                }
                break;
            }
            seen += chunk_total;
        }
    }
}

__global__ void __launch_bounds__(1024)
k_sel_find(const uint32_t* __restrict__ hist, uint64_t k, int round, MaskSelect* __restrict__ sel)
{
    sel_find_body(hist, k, round, sel);
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

// ---------------------------------------------------------------------------------
// The same steps for several clients at once: one job per client with b < 1, the job
// index in blockIdx.y (blockIdx.x for the one-block steps).
// ---------------------------------------------------------------------------------
struct SelJob {
    uint64_t seed, d, k;
    MaskSelect* sel;
    uint32_t* hist;                  // three 2048-bin histograms (one per digit round)
    unsigned long long* chunks;      // one packed count per 1024 coordinates
    const float* in;                 // compact: the client's input row; scatter: its estimate of the kept coordinates
    float* out;                      // compact: the compacted vector
    uint2* cand;                     // two-pass selection: (key, coordinate) of the keys that share tau's first digit
    uint32_t* keep;                  // two-pass selection: the mask as a bitmap (bit i % 32 of word i / 32)
    uint32_t lo, hi;                 // one-pass selection: the band of keys predicted to hold tau (empty if lo > hi)
};

// Batched selection finds the k-th smallest key in three digit rounds of 10, 11 and 11
// bits with histograms of up to 2048 bins (job.hist holds three of them).  Round 0 sees every key,
// so each block counts a long run of keys in shared memory and adds its non-empty bins to
// the global histogram once; rounds 1 and 2 only see the keys that share the digits found
// so far (one in 1024, one in two million) and count them in global memory directly.
// sel->bin_hi carries the digits found so far, sel->below_hi the keys below them.
constexpr int kSelBins = 2048;
constexpr int kSelCallsPerThread = 32;     // Philox calls (4 keys each) per thread and block in a histogram round

__device__ __forceinline__ int sel_digit_shift(int round) { return round == 0 ? 22 : round == 1 ? 11 : 0; }
__device__ __forceinline__ int sel_digit_bits(int round) { return round == 0 ? 10 : 11; }

__global__ void __launch_bounds__(kSelThreads)
k_selb_hist(const SelJob* __restrict__ jobs, int round)
{
    __shared__ uint32_t s_hist[kSelBins];
    const SelJob job = jobs[blockIdx.y];
    uint32_t* hist = job.hist + round * kSelBins;
    const uint64_t calls = (job.d + 3) / 4;
    const uint64_t first = (uint64_t)blockIdx.x * kSelThreads * kSelCallsPerThread;
    if (first >= calls) return;
    const int shift = sel_digit_shift(round);
    const uint32_t mask = (1u << sel_digit_bits(round)) - 1u;
    const uint32_t prefix = round ? job.sel->bin_hi : 0u;
    const int pshift = shift + sel_digit_bits(round);         // bits above this digit
    if (round == 0)
        for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) s_hist[b] = 0u;
    __syncthreads();
    for (int it = 0; it < kSelCallsPerThread; ++it) {
        const uint64_t t = first + (uint64_t)it * kSelThreads + threadIdx.x;
        if (t >= calls) break;
        const uint4 k4 = mask_keys(job.seed, t);
        const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (t * 4 + j >= job.d) break;
            if (round == 0) atomicAdd(&s_hist[keys[j] >> shift], 1u);
            else if ((keys[j] >> pshift) == prefix) atomicAdd(&hist[(keys[j] >> shift) & mask], 1u);
        }
    }
    if (round == 0) {
        __syncthreads();
        for (int b = threadIdx.x; b < kSelBins; b += kSelThreads)
            if (s_hist[b]) atomicAdd(&hist[b], s_hist[b]);
    }
}

// One block per job: the bin of the current round's histogram that holds rank
// k - 1 - (keys below the digits found so far); extends the digits, and after the last
// round writes tau, below and rem.
__global__ void __launch_bounds__(1024)
k_selb_find(const SelJob* __restrict__ jobs, int round)
{
    __shared__ uint32_t warp_total[32];
    __shared__ uint32_t warp_before[32];
    const SelJob job = jobs[blockIdx.x];
    MaskSelect* sel = job.sel;
    const uint32_t* hist = job.hist + round * kSelBins;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t below_so_far = round ? sel->below_hi : 0u;
    const uint32_t prefix = round ? sel->bin_hi : 0u;
    const uint32_t r = (uint32_t)(job.k - 1) - below_so_far;
    // warp w owns bins [64 w, 64 w + 64)
    const uint32_t* run = hist + warp * 64;
    uint32_t v[2], mine = 0;
#pragma unroll
    for (int i = 0; i < 2; ++i) { v[i] = run[i * 32 + lane]; mine += v[i]; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if (lane == 0) warp_total[warp] = mine;
    __syncthreads();
    if (warp == 0) {
        const uint32_t w = warp_total[lane];
        uint32_t inc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += t;
        }
        warp_before[lane] = inc - w;
    }
    __syncthreads();
    const uint32_t before = warp_before[warp];
    if (r >= before && r < before + warp_total[warp]) {        // exactly one warp
        uint32_t seen = before;
        for (int i = 0; i < 2; ++i) {
            uint32_t inc = v[i];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, inc, o);
                if (lane >= o) inc += t;
            }
            const uint32_t chunk_total = __shfl_sync(0xffffffffu, inc, 31);
            if (r < seen + chunk_total) {
                const uint32_t hit = __ballot_sync(0xffffffffu, r < seen + inc);
                const int firstl = __ffs(hit) - 1;
                if (lane == firstl) {
                    const uint32_t bin = (uint32_t)(warp * 64 + i * 32 + lane);
                    const uint32_t below = below_so_far + seen + inc - v[i];
                    const uint32_t digits = (prefix << sel_digit_bits(round)) | bin;
                    if (round < 2) {
                        sel->bin_hi = digits;
                        sel->below_hi = below;
                    } else {
                        sel->tau = digits;
                        sel->below = below;
                        sel->rem = (uint32_t)job.k - below;        // ties to keep, >= 1
                    }
                }
                break;
            }
            seen += chunk_total;
        }
    }
}

__global__ void __launch_bounds__(kSelThreads)
k_selb_chunk_count(const SelJob* __restrict__ jobs)
{
    __shared__ unsigned long long scratch[33];
    const SelJob job = jobs[blockIdx.y];
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t cls[4];
    const unsigned long long mine = classify4(job.seed, t, job.d, job.sel->tau, cls);
    unsigned long long total;
    block_exclusive_scan(mine, scratch, &total);
    if (threadIdx.x == 0) job.chunks[blockIdx.x] = total;
}

__global__ void __launch_bounds__(1024)
k_selb_chunk_scan(const SelJob* __restrict__ jobs, uint64_t n_chunks)
{
    __shared__ unsigned long long scratch[33];
    unsigned long long* chunk_counts = jobs[blockIdx.x].chunks;
    const uint64_t per = (n_chunks + blockDim.x - 1) / blockDim.x;
    const uint64_t lo = min((uint64_t)threadIdx.x * per, n_chunks), hi = min(lo + per, n_chunks);
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

// ---------------------------------------------------------------------------------
// Selection with a candidate list (vectors short enough for it, kSelCandCap).
//
// Keys below a band [lo, hi] that is known to hold tau are kept whatever tau's exact value
// is: one pass over the keys counts them per chunk of 1024 coordinates and marks them in
// the job's mask bitmap, and appends the keys inside the band to the job's candidate list
// with their coordinates.  One block per job then finds tau among the candidates alone and,
// for each candidate that is kept (below tau, or equal to it and among the first `rem` such
// coordinates), sets its bit and adds it to its chunk's count.  Compaction and scatter read
// the bitmap.  job.hist[kSelBins] counts the candidates (zeroed with the histograms).
//
// Where the band comes from:
//  * predicted (the default): the keys are uniform, so the k-th smallest of d is close to
//    (k/d) 2^32; the host puts a band of a few standard deviations around it and the keys
//    are generated once per side.  If tau turns out to lie outside (or the list overflows)
//    the job is flagged and k_selc_redo does it again the second way, one block per job:
//    slow, but it runs about once in 10^4 jobs, and the mask is the same either way.
//  * from a histogram round: the bin of tau's top 11 bits (one key in 2048 is a candidate);
//    the keys are generated twice per side.
// ---------------------------------------------------------------------------------
constexpr int kSelFirstShift = 21;                     // first digit = key >> 21 (11 bits, kSelBins bins)
constexpr uint32_t kSelCandCap = 61440;                // candidates a job can hold (480 KB)
constexpr uint32_t kStatusScratch = 0x10u;             // EDEN_STATUS_SCRATCH
constexpr int kSelDigitBins = 4096;                    // bins of a digit round among the candidates

__global__ void __launch_bounds__(kSelThreads)
k_selc_hist(const SelJob* __restrict__ jobs)
{
    __shared__ uint32_t s_hist[kSelBins];
    const SelJob job = jobs[blockIdx.y];
    const uint64_t calls = (job.d + 3) / 4;
    const uint64_t first = (uint64_t)blockIdx.x * kSelThreads * kSelCallsPerThread;
    if (first >= calls) return;
    for (int b = threadIdx.x; b < kSelBins; b += kSelThreads) s_hist[b] = 0u;
    __syncthreads();
    for (int it = 0; it < kSelCallsPerThread; ++it) {
        const uint64_t t = first + (uint64_t)it * kSelThreads + threadIdx.x;
        if (t >= calls) break;
        const uint4 k4 = mask_keys(job.seed, t);
        const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (t * 4 + j < job.d) atomicAdd(&s_hist[keys[j] >> kSelFirstShift], 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kSelBins; b += kSelThreads)
        if (s_hist[b]) atomicAdd(&job.hist[b], s_hist[b]);
}

// One warp, one chunk of 1024 coordinates: lane l takes the eight Philox calls of the
// chunk's bitmap word l, builds the word in a register, and the warp adds up the counts;
// nothing goes through shared memory or a block barrier.
__device__ __forceinline__ void collect_chunk(const SelJob& job, uint64_t chunk, uint32_t lo, uint32_t hi)
{
    const uint32_t lane = threadIdx.x & 31u;
    const bool empty = lo > hi;
    const uint32_t span = hi - lo;
    uint32_t word = 0u;
    const uint64_t t0 = chunk * (kSelChunk / 4) + lane * 8u;
    if (t0 * 4 + 32 <= job.d) {
        // all 32 coordinates exist: no bounds checks, and four Philox calls at a time with
        // nothing between them, so that their multiply chains interleave
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            uint4 k4[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) k4[c] = mask_keys(job.seed, t0 + 4 * half + c);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const uint32_t keys[4] = {k4[c].x, k4[c].y, k4[c].z, k4[c].w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int bit = 16 * half + 4 * c + j;
                    word |= (keys[j] < lo ? 1u : 0u) << bit;
                    if (keys[j] - lo <= span && !empty) {
                        const uint32_t slot = atomicAdd(&job.hist[kSelBins], 1u);
                        if (slot < kSelCandCap) job.cand[slot] = make_uint2(keys[j], (uint32_t)(t0 * 4) + bit);
                    }
                }
            }
        }
    } else {
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
            const uint64_t t = t0 + c;
            if (t * 4 >= job.d) break;
            const uint4 k4 = mask_keys(job.seed, t);
            const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint64_t i = t * 4 + j;
                if (i >= job.d) break;
                if (keys[j] < lo) {
                    word |= 1u << (4 * c + j);
                } else if (keys[j] <= hi && !empty) {
                    const uint32_t slot = atomicAdd(&job.hist[kSelBins], 1u);
                    if (slot < kSelCandCap) job.cand[slot] = make_uint2(keys[j], (uint32_t)i);
                }
            }
        }
    }
    job.keep[chunk * 32u + lane] = word;
    const uint32_t count = __reduce_add_sync(0xffffffffu, (uint32_t)__popc(word));
    if (lane == 0) job.chunks[chunk] = count;
}

// PREDICTED: the band is job.lo .. job.hi; otherwise the bin of the digit in sel->bin_hi.
template <bool PREDICTED>
__global__ void __launch_bounds__(kSelThreads)
k_selc_collect(const SelJob* __restrict__ jobs, uint64_t n_chunks)
{
    const SelJob job = jobs[blockIdx.y];
    const uint64_t chunk = (uint64_t)blockIdx.x * (kSelThreads / 32) + (threadIdx.x >> 5);
    if (chunk >= n_chunks) return;
    const uint32_t lo = PREDICTED ? job.lo : job.sel->bin_hi << kSelFirstShift;
    const uint32_t hi = PREDICTED ? job.hi : lo | ((1u << kSelFirstShift) - 1u);
    collect_chunk(job, chunk, lo, hi);
}

// A block's walk over a job's candidate list, eight loads in flight per thread (one block
// per job: the walk is bound by the latency of the loads, not by their number).
template <class F>
__device__ __forceinline__ void for_each_candidate(const SelJob& job, uint32_t n, F f)
{
    for (uint32_t c0 = threadIdx.x; c0 < n; c0 += 8u * blockDim.x) {
        uint2 kc[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const uint32_t c = c0 + u * blockDim.x;
            kc[u] = c < n ? __ldcg(&job.cand[c]) : make_uint2(0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
            if (c0 + u * blockDim.x < n) f(kc[u]);
    }
}

// Sum of the job's chunk counts (SCAN: replaced in place by their exclusive prefix sums),
// thread t taking a contiguous run, eight loads in flight.  Whole block.
template <bool SCAN>
__device__ __forceinline__ unsigned long long chunk_counts_sum(const SelJob& job, uint64_t n_chunks,
                                                               unsigned long long* scan_scratch)
{
    const uint64_t per = (n_chunks + blockDim.x - 1) / blockDim.x;
    const uint64_t c0 = min((uint64_t)threadIdx.x * per, n_chunks), c1 = min(c0 + per, n_chunks);
    unsigned long long mine = 0;
    for (uint64_t j0 = c0; j0 < c1; j0 += 8) {
        unsigned long long v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = j0 + u < c1 ? __ldcg(&job.chunks[j0 + u]) : 0ull;
#pragma unroll
        for (int u = 0; u < 8; ++u) mine += v[u];
    }
    unsigned long long total;
    unsigned long long run = block_exclusive_scan(mine, scan_scratch, &total);
    if (SCAN) {
        for (uint64_t j0 = c0; j0 < c1; j0 += 8) {
            unsigned long long v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = j0 + u < c1 ? __ldcg(&job.chunks[j0 + u]) : 0ull;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (j0 + u < c1) job.chunks[j0 + u] = run;
                run += v[u];
            }
        }
    }
    return total;
}

// Scratch of the block that resolves a job (1024 threads).
struct ResolveShared {
    uint32_t hist[kSelDigitBins];
    unsigned long long scan[33];
    uint32_t ties[256];
    uint32_t bin, before, n_ties;
};

// Finds tau among the job's n candidates, all of which lie in [base, base + 2^width), given
// that `below` keys are smaller than every candidate; marks the kept candidates; scans the
// chunk counts into positions.  The offset of tau inside the band is settled from the top
// in one to three digits of at most 12 bits each.  Whole block, 1024 threads.
__device__ __forceinline__ void resolve_job(const SelJob& job, ResolveShared& sh, uint32_t n, uint32_t base,
                                            int width, uint32_t below, uint64_t n_chunks)
{
    MaskSelect* sel = job.sel;
    const int rounds = (width + 11) / 12;
    const int per_round = rounds ? (width + rounds - 1) / rounds : 0;
    uint32_t prefix = 0u;                              // the bits of tau - base fixed so far
    int fixed = 0;                                     // how many they are
    while (fixed < width) {
        const int bits = width - fixed < per_round ? width - fixed : per_round;
        const int shift = width - fixed - bits;
        for (int b = threadIdx.x; b < kSelDigitBins; b += blockDim.x) sh.hist[b] = 0u;
        if (threadIdx.x == 0) { sh.bin = 0u; sh.before = 0u; }
        __syncthreads();
        for_each_candidate(job, n, [&](uint2 kc) {
            const uint32_t rel = kc.x - base;
            if (fixed == 0 || (rel >> (shift + bits)) == prefix)
                atomicAdd(&sh.hist[(rel >> shift) & ((1u << bits) - 1u)], 1u);
        });
        __syncthreads();
        // thread t owns bins 4t .. 4t + 3; the rank looked for is k - 1 - below
        const uint32_t r = (uint32_t)(job.k - 1) - below;
        uint32_t v[4], mine = 0u;
#pragma unroll
        for (int i = 0; i < 4; ++i) { v[i] = sh.hist[4 * threadIdx.x + i]; mine += v[i]; }
        unsigned long long total;
        uint32_t before = (uint32_t)block_exclusive_scan((unsigned long long)mine, sh.scan, &total);
        if (r >= before && r < before + mine) {        // exactly one thread
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                if (r >= before && r < before + v[i]) {
                    sh.bin = 4 * threadIdx.x + i;
                    sh.before = before;
                }
                before += v[i];
            }
        }
        __syncthreads();
        prefix = (prefix << bits) | sh.bin;
        below += sh.before;
        fixed += bits;
        __syncthreads();
    }
    const uint32_t tau = base + prefix;
    const uint32_t rem = (uint32_t)job.k - below;      // ties to keep, >= 1
    if (threadIdx.x == 0) {
        sel->tau = tau;
        sel->below = below;
        sel->rem = rem;
        sh.n_ties = 0u;
    }
    __syncthreads();
    // the candidates that are kept: below tau, or equal to it with fewer than `rem` equal
    // keys at smaller coordinates.  Equal keys are rare, so their coordinates are gathered
    // in shared memory and ranked there; a list that does not fit is ranked in place.
    constexpr uint32_t kTieCap = 256;
    for_each_candidate(job, n, [&](uint2 kc) {
        if (kc.x < tau) {
            atomicOr(&job.keep[kc.y >> 5], 1u << (kc.y & 31u));
            atomicAdd(&job.chunks[kc.y >> 10], 1ull);
        } else if (kc.x == tau) {
            const uint32_t slot = atomicAdd(&sh.n_ties, 1u);
            if (slot < kTieCap) sh.ties[slot] = kc.y;
        }
    });
    __syncthreads();
    const uint32_t n_ties = sh.n_ties;
    if (n_ties <= kTieCap) {
        for (uint32_t i = threadIdx.x; i < n_ties; i += blockDim.x) {
            const uint32_t coord = sh.ties[i];
            uint32_t before = 0;
            for (uint32_t o = 0; o < n_ties; ++o) before += sh.ties[o] < coord ? 1u : 0u;
            if (before < rem) {
                atomicOr(&job.keep[coord >> 5], 1u << (coord & 31u));
                atomicAdd(&job.chunks[coord >> 10], 1ull);
            }
        }
    } else {
        for (uint32_t c = threadIdx.x; c < n; c += blockDim.x) {
            const uint2 kc = job.cand[c];
            if (kc.x != tau) continue;
            uint32_t before = 0;
            for (uint32_t o = 0; o < n; ++o) {
                const uint2 ko = job.cand[o];
                before += (ko.x == tau && ko.y < kc.y) ? 1u : 0u;
            }
            if (before < rem) {
                atomicOr(&job.keep[kc.y >> 5], 1u << (kc.y & 31u));
                atomicAdd(&job.chunks[kc.y >> 10], 1ull);
            }
        }
    }
    // every count is final: scan them in place (reads from L2, where the atomics landed)
    __syncthreads();
    chunk_counts_sum<true>(job, n_chunks, sh.scan);
}

// One block of 1024 threads per job, behind k_selc_collect.  PREDICTED: the keys below the
// band are the sum of the chunk counts; the prediction holds if the list did not overflow
// and the rank looked for falls among the candidates.  If it does not, the job is flagged
// for k_selc_redo and its candidate counter is cleared.
template <bool PREDICTED>
__global__ void __launch_bounds__(1024)
k_selc_resolve(const SelJob* __restrict__ jobs, uint32_t* __restrict__ status, uint64_t n_chunks)
{
    __shared__ ResolveShared sh;
    const SelJob job = jobs[blockIdx.x];
    MaskSelect* sel = job.sel;
    const uint32_t found = job.hist[kSelBins];
    if (!PREDICTED) {
        if (found > kSelCandCap && threadIdx.x == 0) atomicOr(status, kStatusScratch);
        resolve_job(job, sh, min(found, kSelCandCap), sel->bin_hi << kSelFirstShift, kSelFirstShift, sel->below_hi,
                    n_chunks);
        return;
    }
    const unsigned long long total = chunk_counts_sum<false>(job, n_chunks, sh.scan);
    const bool holds = found <= kSelCandCap && job.k >= 1 && total <= job.k - 1 && job.k - 1 - total < (uint64_t)found;
    if (!holds) {
        if (threadIdx.x == 0) {
            sel->fallback = 1u;
            job.hist[kSelBins] = 0u;
        }
        return;
    }
    resolve_job(job, sh, found, job.lo, 32 - __clz(job.hi - job.lo), (uint32_t)total, n_chunks);
}

// The jobs whose prediction failed, one block of 1024 threads per job, every step of the
// histogram form inside the block: first-digit histogram over all keys, the digit that holds
// rank k - 1, the collecting pass, the candidates.  Every other job returns at once.
__global__ void __launch_bounds__(1024)
k_selc_redo(const SelJob* __restrict__ jobs, uint32_t* __restrict__ status, uint64_t n_chunks)
{
    __shared__ ResolveShared sh;
    const SelJob job = jobs[blockIdx.x];
    MaskSelect* sel = job.sel;
    if (!sel->fallback) return;
    static_assert(kSelBins <= kSelDigitBins, "the first-digit histogram uses the resolve scratch");
    for (int b = threadIdx.x; b < kSelBins; b += blockDim.x) sh.hist[b] = 0u;
    if (threadIdx.x == 0) { sh.bin = 0u; sh.before = 0u; }
    __syncthreads();
    const uint64_t calls = (job.d + 3) / 4;
    for (uint64_t t = threadIdx.x; t < calls; t += blockDim.x) {
        const uint4 k4 = mask_keys(job.seed, t);
        const uint32_t keys[4] = {k4.x, k4.y, k4.z, k4.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (t * 4 + j < job.d) atomicAdd(&sh.hist[keys[j] >> kSelFirstShift], 1u);
    }
    __syncthreads();
    {
        // thread t owns bins 2t and 2t + 1
        const uint32_t r = (uint32_t)(job.k - 1);
        const uint32_t v0 = sh.hist[2 * threadIdx.x], v1 = sh.hist[2 * threadIdx.x + 1];
        unsigned long long total;
        const uint32_t before = (uint32_t)block_exclusive_scan((unsigned long long)(v0 + v1), sh.scan, &total);
        if (r >= before && r < before + v0 + v1) {     // exactly one thread (none if k = 0)
            const bool second = r >= before + v0;
            sh.bin = 2 * threadIdx.x + (second ? 1u : 0u);
            sh.before = before + (second ? v0 : 0u);
        }
        __syncthreads();
    }
    const uint32_t digit = sh.bin, below = sh.before;
    if (threadIdx.x == 0) {
        sel->bin_hi = digit;
        sel->below_hi = below;
    }
    const uint32_t lo = digit << kSelFirstShift, hi = lo | ((1u << kSelFirstShift) - 1u);
    for (uint64_t chunk = threadIdx.x >> 5; chunk < n_chunks; chunk += blockDim.x >> 5)
        collect_chunk(job, chunk, lo, hi);
    __threadfence();
    __syncthreads();
    const uint32_t found = __ldcg(&job.hist[kSelBins]);
    if (found > kSelCandCap && threadIdx.x == 0) atomicOr(status, kStatusScratch);
    resolve_job(job, sh, min(found, kSelCandCap), lo, kSelFirstShift, below, n_chunks);
}

// One warp walks one chunk of 1024 coordinates in eight pieces of 128, lane l taking the
// four coordinates 128 i + 4 l .. + 3 of piece i, so that the vector accesses of a piece are
// one contiguous 512 bytes.  Lane l also holds the chunk's bitmap word l; a shuffle scan of
// the population counts gives the kept coordinates before each word.
struct ChunkMask {
    uint32_t word;      // bitmap word `lane` of the chunk
    uint32_t before;    // kept coordinates of the chunk in the words below it
};

__device__ __forceinline__ ChunkMask chunk_mask(const uint32_t* __restrict__ keep, uint64_t chunk)
{
    const uint32_t lane = threadIdx.x & 31u;
    ChunkMask m;
    m.word = keep[chunk * 32u + lane];
    uint32_t inc = (uint32_t)__popc(m.word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= (uint32_t)o) inc += v;
    }
    m.before = inc - (uint32_t)__popc(m.word);
    return m;
}

// The lane's four mask bits in piece i and the position, among the chunk's kept coordinates,
// of the first of them that is kept.
__device__ __forceinline__ uint32_t piece_position(const ChunkMask& m, int i, uint32_t& nibble)
{
    const uint32_t lane = threadIdx.x & 31u;
    const int w = 4 * i + (int)(lane >> 3);                       // the word that holds the lane's nibble
    const uint32_t word = __shfl_sync(0xffffffffu, m.word, w);
    const uint32_t before = __shfl_sync(0xffffffffu, m.before, w);
    const uint32_t shift = 4u * (lane & 7u);
    nibble = (word >> shift) & 0xFu;
    return before + (uint32_t)__popc(word & ((1u << shift) - 1u));
}

// Sender: y_c[pos] = x_c[i] for the kept coordinates of every job, from the bitmap.
__global__ void __launch_bounds__(kSelThreads)
k_selc_compact(const SelJob* __restrict__ jobs, uint64_t n_chunks)
{
    const SelJob job = jobs[blockIdx.y];
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t chunk = (uint64_t)blockIdx.x * (kSelThreads / 32) + (threadIdx.x >> 5);
    if (chunk >= n_chunks) return;
    const uint64_t base = chunk * kSelChunk;
    const bool vec = ((uintptr_t)job.in & 15u) == 0 && base + kSelChunk <= job.d;
    // the whole chunk's input first (eight 16-byte loads in flight per lane), whatever the mask keeps
    float xs[8][4];
    if (vec) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float4 x4 = *reinterpret_cast<const float4*>(job.in + base + 128u * i + 4u * lane);
            xs[i][0] = x4.x; xs[i][1] = x4.y; xs[i][2] = x4.z; xs[i][3] = x4.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint64_t c = base + 128u * i + 4u * lane + j;
                xs[i][j] = c < job.d ? job.in[c] : 0.f;
            }
    }
    const ChunkMask m = chunk_mask(job.keep, chunk);
    float* out = job.out + job.chunks[chunk];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        uint32_t nib;
        uint32_t pos = piece_position(m, i, nib);
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if ((nib >> j) & 1u) out[pos++] = xs[i][j];
    }
}

// Receiver: out[i] += sum over the jobs of yhat_c[pos_c(i)] for the coordinates job c kept
// (Section 4.1: the receiver restores through the same mask).  One pass over out.
__global__ void __launch_bounds__(kSelThreads)
k_selc_scatter(const SelJob* __restrict__ jobs, uint32_t n_jobs, uint64_t d, float* __restrict__ out,
               uint64_t n_chunks)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t chunk = (uint64_t)blockIdx.x * (kSelThreads / 32) + (threadIdx.x >> 5);
    if (chunk >= n_chunks) return;
    const uint64_t base = chunk * kSelChunk;
    float add[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) add[i][j] = 0.f;
    for (uint32_t c = 0; c < n_jobs; ++c) {
        const SelJob job = jobs[c];
        const ChunkMask m = chunk_mask(job.keep, chunk);
        const float* in = job.in + job.chunks[chunk];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            uint32_t nib;
            uint32_t pos = piece_position(m, i, nib);
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if ((nib >> j) & 1u) add[i][j] += in[pos++];
        }
    }
    const bool vec = ((uintptr_t)out & 15u) == 0 && base + kSelChunk <= d;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const uint64_t c0 = base + 128u * i + 4u * lane;
        if (vec) {
            if (add[i][0] != 0.f || add[i][1] != 0.f || add[i][2] != 0.f || add[i][3] != 0.f) {
                float4* p = reinterpret_cast<float4*>(out + c0);
                float4 v = *p;
                v.x += add[i][0]; v.y += add[i][1]; v.z += add[i][2]; v.w += add[i][3];
                *p = v;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (c0 + j < d && add[i][j] != 0.f) out[c0 + j] += add[i][j];
        }
    }
}

// ---------------------------------------------------------------------------------
// Sparsification after the rotation (Section 4.1, the other order): the mask is over the
// rotated coordinates and the message is the one-bit codes of the kept ones, in index
// order.  One warp per chunk of 1024 coordinates (lane l: word l of the chunk's 32 code
// words and 32 bitmap words); job.in is the full code stream, job.out the message
// (sender), or the other way round (receiver); both are word arrays passed through the
// job's float pointers.
// ---------------------------------------------------------------------------------
// the bits of `code` at the set positions of `mask`, packed from bit 0
__device__ __forceinline__ uint32_t bits_extract(uint32_t code, uint32_t mask)
{
    uint32_t out = 0u, n = 0u;
    while (mask) {
        const uint32_t b = mask & (0u - mask);
        out |= (code & b) ? (1u << n) : 0u;
        ++n;
        mask &= mask - 1u;
    }
    return out;
}
// the low bits of `bits`, spread to the set positions of `mask`
__device__ __forceinline__ uint32_t bits_deposit(uint32_t bits, uint32_t mask)
{
    uint32_t out = 0u;
    while (mask) {
        const uint32_t b = mask & (0u - mask);
        out |= (bits & 1u) ? b : 0u;
        bits >>= 1;
        mask &= mask - 1u;
    }
    return out;
}

// words of the full code stream / the bitmap of one job (both cover whole chunks in the
// bitmap; the code stream ends at ceil(d / 32) words)
template <bool PACK>
__global__ void __launch_bounds__(kSelThreads)
k_after_rotation_bits(const SelJob* __restrict__ jobs, uint64_t n_chunks)
{
    const SelJob job = jobs[blockIdx.y];
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t chunk = (uint64_t)blockIdx.x * (kSelThreads / 32) + (threadIdx.x >> 5);
    if (chunk >= n_chunks) return;                                    // whole warps leave together
    const uint64_t w = chunk * 32u + lane;
    const uint64_t code_words = (job.d + 31u) >> 5;
    const uint32_t mask = job.keep[w];
    const uint32_t cnt = (uint32_t)__popc(mask);
    uint32_t inc = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t v = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= (uint32_t)o) inc += v;
    }
    const uint64_t pos = job.chunks[chunk] + (uint64_t)(inc - cnt);   // the message bit of the word's first kept coordinate
    const uint32_t sh = (uint32_t)(pos & 31u);
    if (PACK) {
        const uint32_t* full = reinterpret_cast<const uint32_t*>(job.in);
        uint32_t* msg = reinterpret_cast<uint32_t*>(job.out);
        if (cnt == 0u) return;
        const uint32_t bits = bits_extract(w < code_words ? full[w] : 0u, mask);
        atomicOr(&msg[pos >> 5], bits << sh);                         // the message was cleared before
        if (sh + cnt > 32u) atomicOr(&msg[(pos >> 5) + 1], bits >> (32u - sh));
    } else {
        const uint32_t* msg = reinterpret_cast<const uint32_t*>(job.in);
        uint32_t* full = reinterpret_cast<uint32_t*>(job.out);
        uint32_t bits = 0u;
        if (cnt) {
            const uint32_t lo = msg[pos >> 5];
            const uint32_t hi = sh + cnt > 32u ? msg[(pos >> 5) + 1] : 0u;
            bits = __funnelshift_r(lo, hi, sh);
        }
        if (w < code_words) full[w] = bits_deposit(bits, mask);
    }
}

// Sender: y_c[pos] = x_c[i] for the kept coordinates of every job.
__global__ void __launch_bounds__(kSelThreads)
k_selb_compact(const SelJob* __restrict__ jobs)
{
    __shared__ unsigned long long scratch[33];
    const SelJob job = jobs[blockIdx.y];
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const uint32_t tau = job.sel->tau, rem = job.sel->rem;
    uint32_t cls[4];
    const unsigned long long mine = classify4(job.seed, t, job.d, tau, cls);
    unsigned long long total;
    const unsigned long long before = block_exclusive_scan(mine, scratch, &total) + job.chunks[blockIdx.x];
    uint32_t below = (uint32_t)before, ties = (uint32_t)(before >> 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t i = t * 4 + j;
        const bool keep = cls[j] == 1 || (cls[j] == 2 && ties < rem);
        if (keep) job.out[(uint64_t)below + min(ties, rem)] = job.in[i];
        if (cls[j] == 1) ++below;
        if (cls[j] == 2) ++ties;
    }
}

// Receiver: out[i] += sum over the jobs of yhat_c[pos_c(i)] for the coordinates job c kept
// (Section 4.1: the receiver restores through the same mask).  One pass over out.
__global__ void __launch_bounds__(kSelThreads)
k_selb_scatter(const SelJob* __restrict__ jobs, uint32_t n_jobs, uint64_t d, float* __restrict__ out)
{
    __shared__ unsigned long long scratch[33];
    const uint64_t t = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    float add[4] = {0.f, 0.f, 0.f, 0.f};
    for (uint32_t c = 0; c < n_jobs; ++c) {
        const SelJob job = jobs[c];
        const uint32_t tau = job.sel->tau, rem = job.sel->rem;
        uint32_t cls[4];
        const unsigned long long mine = classify4(job.seed, t, d, tau, cls);
        unsigned long long total;
        const unsigned long long before = block_exclusive_scan(mine, scratch, &total) + job.chunks[blockIdx.x];
        uint32_t below = (uint32_t)before, ties = (uint32_t)(before >> 32);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const bool keep = cls[j] == 1 || (cls[j] == 2 && ties < rem);
            if (keep) add[j] += job.in[(uint64_t)below + min(ties, rem)];
            if (cls[j] == 1) ++below;
            if (cls[j] == 2) ++ties;
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t i = t * 4 + j;
        if (i < d && add[j] != 0.f) out[i] += add[j];
    }
}

}  // namespace eden
