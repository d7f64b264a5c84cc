// Register-blocked transform kernels for rotation dimensions of 2^14 and more.
//
// Every kernel works on a tile of 8192 floats with 256 threads, 32 values per thread,
// two to five resident blocks per SM (set per kernel).  Butterflies run in registers as packed fp32 pairs
// (add.rn.f32x2 / sub.rn.f32x2: one instruction per two coordinates); between register
// steps the tile is transposed through shared memory with 64- or 128-bit conflict-free
// accesses; global loads and stores are 64- or 128-bit and fully coalesced.
//
//  * column pass (k_f_col: the sender's first pass and the in-place middle passes;
//    k_f_dec_last: the receiver's last pass): the tile is 2^LR rows of
//    8192/2^LR consecutive coordinates, rows 2^lo apart; the LR row bits are transformed.
//    Values travel as float4 (four neighbouring columns), so every stage is two packed
//    instructions per float4 pair.
//  * row pass (k_f_enc_last, k_f_dec_first): the tile is 8192 consecutive coordinates; all
//    13 index bits are transformed in three register steps (5 + 4 + 4 bits) on float2
//    units.  At the message side of the pass a thread owns 32 consecutive coordinates, so
//    it builds (or reads) whole 32-bit code words by itself.
//  * thread-block clusters (template parameter LC > 0): 2^LC blocks of a cluster hold 2^LC
//    tiles that differ in the LC index bits just above the block's own; those stages are
//    done by one exchange through distributed shared memory: every block fetches its
//    1/2^LC slice of all tiles of the cluster, does the LC stages in registers and writes
//    the results where they belong.  That transforms 2^24 .. 2^27 coordinates in two
//    sweeps over HBM instead of three, but on B200 the two cluster barriers per tile cost
//    more than the sweep they save, so the default plan launches every kernel with LC = 0
//    and the cluster forms are a tuning option.
#pragma once
#include "eden_device.cuh"
#include "kernels_generic.cuh"
#include <cooperative_groups.h>

namespace eden {

constexpr int kFastThreads = 256;
constexpr int kFastTileLog = 13;
constexpr int kFastMaxColBits = 8;     // row bits one block transforms in a column pass
constexpr int kFastClusterLog = 3;     // a cluster of 8 blocks adds three more bits to a pass

namespace cg = cooperative_groups;

// Cluster barrier that publishes this block's shared-memory writes to the other blocks
// of the cluster: the block-wide barrier orders every thread's writes before thread 0,
// whose cluster-scope fence and (relaxed) arrival form the release; every thread's wait
// acquires.  One fence per block instead of one per thread.
__device__ __forceinline__ void cluster_sync_publish()
{
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("fence.acq_rel.cluster;" ::: "memory");
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Cluster barrier that only orders execution: callers use it after they have consumed
// every value they read from other blocks' shared memory, to tell the owners that the
// memory may be overwritten.
__device__ __forceinline__ void cluster_sync_execution()
{
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.aligned;" ::: "memory");
}

typedef unsigned long long u64;

// 32-bit shared-memory address of a pointer into shared memory
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// ---------------------------------------------------------------------------------
// packed fp32 pairs
// ---------------------------------------------------------------------------------
__device__ __forceinline__ u64 pack2(float lo, float hi)
{
    u64 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(u64 v, float& lo, float& hi)
{
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
// (a, b) -> (a + b, a - b) on both halves
__device__ __forceinline__ void bfly2(u64& a, u64& b)
{
    u64 s, d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(s) : "l"(a), "l"(b));
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    a = s;
    b = d;
}
// butterfly between the two halves of one pair: (x, y) -> (x + y, x - y)
__device__ __forceinline__ u64 bfly_inner(u64 v)
{
    float x, y;
    unpack2(v, x, y);
    return pack2(x + y, x - y);
}
__device__ __forceinline__ u64 fma2(u64 a, u64 b, u64 c)
{
    u64 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// flips the sign of each half where the matching bit of `bits` (bit 0 -> lo, bit 1 -> hi) is set
__device__ __forceinline__ u64 flip2(u64 v, uint32_t bits)
{
    float lo, hi;
    unpack2(v, lo, hi);
    lo = __uint_as_float(__float_as_uint(lo) ^ (bits << 31));
    hi = __uint_as_float(__float_as_uint(hi) ^ ((bits << 30) & 0x80000000u));
    return pack2(lo, hi);
}

// Butterflies over the register index bits [0, NB) of 8 float4 values (as 16 packed pairs:
// v[2*k], v[2*k+1] are the halves of float4 k).  Only the top `nb_live` of the NB = 3 index
// bits are transformed (bits below belong to columns).
template <int LIVE>
__device__ __forceinline__ void col_step(u64 (&v)[16])
{
#pragma unroll
    for (int b = 3 - LIVE; b < 3; ++b) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            if (!(k & (1 << b))) {
                bfly2(v[2 * k], v[2 * (k | (1 << b))]);
                bfly2(v[2 * k + 1], v[2 * (k | (1 << b)) + 1]);
            }
        }
    }
}

// ---------------------------------------------------------------------------------
// Column-pass tile: float4 index q in [0, 2048); row = q >> (11 - LR).  Three register
// arrangements (thread -> the 8 float4 it holds), arrangement s holding q bits
// [10-3s, 8-3s] in registers:
//   0: q = t + 256 k                         (coalesced; used for all global traffic in)
//   1: q = (t >> 5) << 8 | k << 5 | (t & 31)
//   2: q = (t >> 2) << 5 | k << 2 | (t & 3)
// Shared memory holds float4 q at f(q) = q ^ (bit 5 of q) << 2, which makes the 128-bit
// accesses of all three arrangements conflict-free.
// ---------------------------------------------------------------------------------
template <int ARR>
__device__ __forceinline__ int col_q(int t, int k)
{
    if (ARR == 0) return t + 256 * k;
    if (ARR == 1) return ((t >> 5) << 8) | (k << 5) | (t & 31);
    return ((t >> 2) << 5) | (k << 2) | (t & 3);
}
__device__ __forceinline__ int col_swz(int q) { return q ^ (((q >> 5) & 1) << 2); }

template <int FROM, int TO>
__device__ __forceinline__ void col_exchange(u64 (&v)[16], ulonglong2* s)
{
    const int t = threadIdx.x;
#pragma unroll
    for (int k = 0; k < 8; ++k) s[col_swz(col_q<FROM>(t, k))] = make_ulonglong2(v[2 * k], v[2 * k + 1]);
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const ulonglong2 w = s[col_swz(col_q<TO>(t, k))];
        v[2 * k] = w.x;
        v[2 * k + 1] = w.y;
    }
}

// number of register steps of a column pass and the arrangement it ends in
template <int LR> struct ColSteps { static constexpr int n = (LR + 2) / 3; static constexpr int last = n - 1; };

// All LR row stages of a column tile held in arrangement 0; returns in arrangement
// ColSteps<LR>::last.  `s` is a 32 KB shared buffer.  The caller must __syncthreads()
// before reusing `s` after this returns (the last read of `s` may still be in flight in
// other warps).
template <int LR>
__device__ __forceinline__ void col_transform(u64 (&v)[16], ulonglong2* s)
{
    col_step<(LR >= 3 ? 3 : LR)>(v);
    if (LR > 3) {
        col_exchange<0, 1>(v, s);
        col_step<(LR >= 6 ? 3 : LR - 3)>(v);
    }
    if (LR > 6) {
        __syncthreads();
        col_exchange<1, 2>(v, s);
        col_step<LR - 6>(v);
    }
}

struct ColTile {
    uint64_t base;      // global index of float 0 of row 0 of this block's tile
    uint64_t base0;     // the same for the tile of cluster rank 0
    uint64_t rank_step; // distance between the tiles of consecutive cluster ranks
    int lo;             // log2 of the distance between rows (in floats)
    int rank;           // this block's rank in its cluster
};

// Tile of block blockIdx.x for a pass over index bits [lo, lo + LR + LC): the block's rows
// are bits [lo, lo + LR); bits [lo + LR, lo + LR + LC) are the cluster rank.
template <int LR, int LC>
__device__ __forceinline__ ColTile col_tile(uint64_t block, int lo)
{
    constexpr int LWC = kFastTileLog - LR;            // log2 columns per row
    const int chunk_bits = lo - LWC;
    const uint64_t super = block >> LC;
    const uint64_t outer = super >> chunk_bits;
    const uint64_t chunk = super & ((1ull << chunk_bits) - 1);
    ColTile ct;
    ct.rank = (int)(block & ((1u << LC) - 1));
    ct.rank_step = 1ull << (lo + LR);
    ct.base0 = (outer << (lo + LR + LC)) + (chunk << LWC);
    ct.base = ct.base0 + (uint64_t)ct.rank * ct.rank_step;
    ct.lo = lo;
    return ct;
}

// offset (in floats) of component 0 of float4 q inside a tile
template <int LR>
__device__ __forceinline__ uint64_t col_offset(const ColTile& ct, int q)
{
    constexpr int LCQ = 11 - LR;                      // log2 float4 per row
    const uint64_t r = (uint64_t)(q >> LCQ);
    const uint64_t cq = (uint64_t)(q & ((1 << LCQ) - 1));
    return (r << ct.lo) + (cq << 2);
}

// The 256 sign words (32 coordinates each) of the block's column tile, word w =
// row * (Wc/32) + j, computed by the first warps into shared memory (one Philox call
// yields the four words of 128 consecutive coordinates).
template <int LR>
__device__ __forceinline__ void col_sign_words(uint64_t seed, const ColTile& ct, uint32_t* s_sign)
{
    constexpr int LWR = kFastTileLog - LR - 5;        // log2 words per row (Wc / 32)
    constexpr int CALLS = LWR >= 2 ? 64 : (LWR == 1 ? 128 : 256);
    const int t = threadIdx.x;
    if (t < CALLS) {
        if (LWR >= 2) {
            // call t covers words 4t .. 4t+3 of the tile (same row: rows hold >= 4 words)
            const int w0 = 4 * t;
            const uint64_t r = (uint64_t)(w0 >> LWR);
            const uint64_t g = (ct.base + (r << ct.lo)) / 32 + (uint64_t)(w0 & ((1 << LWR) - 1));
            const uint4 p = philox_stream(seed, 0u, g >> 2);
            s_sign[w0] = p.x; s_sign[w0 + 1] = p.y; s_sign[w0 + 2] = p.z; s_sign[w0 + 3] = p.w;
        } else if (LWR == 1) {
            // rows hold two words: half a call per row
            const int w0 = 2 * t;
            const uint64_t g = (ct.base + ((uint64_t)t << ct.lo)) / 32;
            const uint4 p = philox_stream(seed, 0u, g >> 2);
            const bool upper = (g & 2) != 0;
            s_sign[w0] = upper ? p.z : p.x;
            s_sign[w0 + 1] = upper ? p.w : p.y;
        } else {
            // rows hold one word: a quarter of a call per row
            const uint64_t g = (ct.base + ((uint64_t)t << ct.lo)) / 32;
            const uint4 p = philox_stream(seed, 0u, g >> 2);
            const uint32_t w = (uint32_t)g & 3u;
            s_sign[t] = w == 0 ? p.x : w == 1 ? p.y : w == 2 ? p.z : p.w;
        }
    }
}

// the four sign bits of float4 q of the tile
template <int LR>
__device__ __forceinline__ uint32_t col_sign_nibble(const uint32_t* s_sign, int q)
{
    constexpr int LCQ = 11 - LR;
    const int r = q >> LCQ, cq = q & ((1 << LCQ) - 1);
    const uint32_t w = s_sign[(LCQ >= 3 ? (r << (LCQ - 3)) : r) + (cq >> 3)];
    return (w >> ((cq & 7) * 4)) & 0xFu;
}

// ---------------------------------------------------------------------------------
// Cluster stage of a column pass.  In: the block's tile in arrangement ARR.  Out: the
// "slice" arrangement: register float4 k holds float4 q = slice_q(rank, t, k) of the tile
// of cluster rank k >> (3 - LC); the LC stages across the ranks are done.  If s_sign is
// given, nib[k] receives the sign nibble of that float4 from its owner's sign words.
// ---------------------------------------------------------------------------------
template <int LC>
__device__ __forceinline__ int slice_q(int rank, int t, int k)
{
    return rank * (2048 >> LC) + t + 256 * (k & ((8 >> LC) - 1));
}

template <int LR, int LC, int ARR, bool SIGNS>
__device__ __forceinline__ void col_cluster_stage(u64 (&v)[16], ulonglong2* s, const uint32_t* s_sign,
                                                  uint32_t (&nib)[8], int rank)
{
    cg::cluster_group cluster = cg::this_cluster();
    const int t = threadIdx.x;
    __syncthreads();                                   // earlier readers of s are done
#pragma unroll
    for (int k = 0; k < 8; ++k) s[col_swz(col_q<ARR>(t, k))] = make_ulonglong2(v[2 * k], v[2 * k + 1]);
    cluster_sync_publish();                            // every tile of the cluster is in shared memory
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const int owner = k >> (3 - LC);
        const int q = slice_q<LC>(rank, t, k);
        const ulonglong2* rs = cluster.map_shared_rank(s, owner);
        const ulonglong2 w = rs[col_swz(q)];
        v[2 * k] = w.x;
        v[2 * k + 1] = w.y;
        if (SIGNS) nib[k] = col_sign_nibble<LR>(cluster.map_shared_rank(s_sign, owner), q);
    }
    col_step<LC>(v);                                   // the LC stages across the tiles (consumes the fetched values)
    if (SIGNS) {
        uint32_t any = 0u;
#pragma unroll
        for (int k = 0; k < 8; ++k) any |= nib[k];
        asm volatile("" :: "r"(any));                  // the sign nibbles have arrived as well
    }
    cluster_sync_execution();                          // owners may now reuse their shared memory
}

// =================================================================================
// Sender, first pass: x -> sign flip -> ||y||^2 -> top stages -> work
// Middle pass (SIGNED = false): work -> stages -> work, in place.
// =================================================================================
template <int LR, int LC, bool FIRST>
__global__ void __launch_bounds__(kFastThreads, 4)
k_f_col(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states, int lo, int publish_inv,
        uint32_t tile0 /* first tile of this launch (launches that cover a slab of the vector) */)
{
    __shared__ ulonglong2 s[2048];
    __shared__ uint32_t s_sign[256];
    __shared__ double red[32];
    const ClientDesc cd = descs[blockIdx.y];
    const ColTile ct = col_tile<LR, LC>(blockIdx.x + tile0, lo);
    const int t = threadIdx.x;
    const float* __restrict__ src = FIRST ? cd.src : cd.work;
    if (FIRST) col_sign_words<LR>(cd.seed, ct, s_sign);
    u64 v[16];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint64_t i = ct.base + col_offset<LR>(ct, col_q<0>(t, k));
        if (!FIRST || i + 3 < cd.valid) {
            const ulonglong2 w = *reinterpret_cast<const ulonglong2*>(src + i);
            v[2 * k] = w.x;
            v[2 * k + 1] = w.y;
        } else {
            const float x0 = i < cd.valid ? src[i] : 0.f;
            const float x1 = i + 1 < cd.valid ? src[i + 1] : 0.f;
            const float x2 = i + 2 < cd.valid ? src[i + 2] : 0.f;
            v[2 * k] = pack2(x0, x1);
            v[2 * k + 1] = pack2(x2, 0.f);
        }
    }
    if (!FIRST && publish_inv && blockIdx.x + tile0 == 0 && t == 0) {
        // sender's middle pass: ||y||^2 is complete, so one thread per client leaves 1/||y||
        // (0 for a zero or non-finite vector) for the row pass, off every block's critical path
        const double n2 = states[blockIdx.y].norm2;
        states[blockIdx.y].factor = (n2 > 0.0 && n2 < INFINITY) ? (float)(1.0 / sqrt(n2)) : 0.f;
    }
    u64 acc = 0ull;
    if (FIRST) {
#pragma unroll
        for (int k = 0; k < 16; ++k) acc = fma2(v[k], v[k], acc);
        __syncthreads();                               // sign words ready
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t nib = col_sign_nibble<LR>(s_sign, col_q<0>(t, k));
            v[2 * k] = flip2(v[2 * k], nib);
            v[2 * k + 1] = flip2(v[2 * k + 1], nib >> 2);
        }
    }
    col_transform<LR>(v, s);
    constexpr int ARR = ColSteps<LR>::last;
    if (LC == 0) {
#pragma unroll
        for (int k = 0; k < 8; ++k)
            *reinterpret_cast<ulonglong2*>(cd.work + ct.base + col_offset<LR>(ct, col_q<ARR>(t, k))) =
                make_ulonglong2(v[2 * k], v[2 * k + 1]);
    } else {
        uint32_t nib[8];
        col_cluster_stage<LR, LC, ARR, false>(v, s, nullptr, nib, ct.rank);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint64_t i = ct.base0 + (uint64_t)(k >> (3 - LC)) * ct.rank_step +
                               col_offset<LR>(ct, slice_q<LC>(ct.rank, t, k));
            *reinterpret_cast<ulonglong2*>(cd.work + i) = make_ulonglong2(v[2 * k], v[2 * k + 1]);
        }
    }
    if (FIRST) {
        float a0, a1;
        unpack2(acc, a0, a1);
        const double tot = block_sum((double)a0 + (double)a1, red);
        if (t == 0) atomicAdd(&states[blockIdx.y].norm2, tot);
    }
}

// =================================================================================
// Receiver, last pass: for every client of the group finish the inverse transform of the
// tile, apply sign and factor, add into registers; store the sum once (Sections 2.2.2,
// 4.2).  mode: OUT_WRITE / OUT_ACC into out[0, d), OUT_YHAT into the client's own work
// buffer (b < 1: one block row per client), or OUT_PART: block row y sums clients
// [y * n_group, min((y + 1) * n_group, n_members)) into out + y * part_stride.
// =================================================================================
template <int LR, int LC>
// Three resident blocks per SM where the pass has an exchange (more than three row bits):
// the extra warps cover the exchange and the per-client load latency (cfg5's shape, six
// bits: 4990 -> 5520 GB/s at the price of a few spilled registers); two where it has none
// and the registers matter more (cfg4's shape, three bits: 5870 GB/s against 5640).
__global__ void __launch_bounds__(kFastThreads, (LR > 3 ? 3 : 2))
k_f_dec_last(const ClientDesc* __restrict__ descs_in, const ClientState* __restrict__ states_in,
             uint32_t n_group, int lo, float* __restrict__ out, uint64_t d, int mode,
             uint32_t n_members, uint64_t part_stride)
{
    // OUT_YHAT: block row y handles member y alone; OUT_PART: its own run of n_group members
    const uint32_t first = mode == OUT_YHAT ? blockIdx.y : mode == OUT_PART ? blockIdx.y * n_group : 0u;
    if (mode == OUT_YHAT) n_group = 1u;
    if (mode == OUT_PART) n_group = min(n_group, n_members - first);
    const ClientDesc* __restrict__ descs = descs_in + first;
    const ClientState* __restrict__ states = states_in + first;
    __shared__ ulonglong2 s[2048];
    __shared__ uint32_t s_sign[256];
    const ColTile ct = col_tile<LR, LC>(blockIdx.x, lo);
    const int t = threadIdx.x;
    constexpr int ARR = ColSteps<LR>::last;
    u64 acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0ull;
    for (uint32_t c = 0; c < n_group; ++c) {
        const float* __restrict__ work = descs[c].work;
        const uint64_t seed = descs[c].seed;
        const float f = states[c].factor;
        u64 v[16];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const ulonglong2 w =
                *reinterpret_cast<const ulonglong2*>(work + ct.base + col_offset<LR>(ct, col_q<0>(t, k)));
            v[2 * k] = w.x;
            v[2 * k + 1] = w.y;
        }
        __syncthreads();                               // previous client's s / s_sign reads are done
        col_sign_words<LR>(seed, ct, s_sign);
        col_transform<LR>(v, s);
        uint32_t nib[8];
        if (LC == 0) {
            if (LR <= 3) __syncthreads();              // no exchange inside: publish the sign words
#pragma unroll
            for (int k = 0; k < 8; ++k) nib[k] = col_sign_nibble<LR>(s_sign, col_q<ARR>(t, k));
        } else {
            col_cluster_stage<LR, LC, ARR, true>(v, s, s_sign, nib, ct.rank);
        }
        const u64 f2 = pack2(f, f);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            acc[2 * k] = fma2(flip2(v[2 * k], nib[k]), f2, acc[2 * k]);
            acc[2 * k + 1] = fma2(flip2(v[2 * k + 1], nib[k] >> 2), f2, acc[2 * k + 1]);
        }
    }
    const uint64_t limit = mode == OUT_YHAT ? (1ull << descs[0].L) : d;
    float* dst = mode == OUT_YHAT ? descs[0].work : mode == OUT_PART ? out + blockIdx.y * part_stride : out;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const uint64_t i = LC == 0
            ? ct.base + col_offset<LR>(ct, col_q<ARR>(t, k))
            : ct.base0 + (uint64_t)(k >> (3 - LC)) * ct.rank_step + col_offset<LR>(ct, slice_q<LC>(ct.rank, t, k));
        float a[4];
        unpack2(acc[2 * k], a[0], a[1]);
        unpack2(acc[2 * k + 1], a[2], a[3]);
        if (i + 3 < limit) {
            float4* p = reinterpret_cast<float4*>(dst + i);
            if (mode == OUT_ACC) {
                const float4 o = *p;
                a[0] += o.x; a[1] += o.y; a[2] += o.z; a[3] += o.w;
            }
            *p = make_float4(a[0], a[1], a[2], a[3]);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (i + e < limit) {
                    if (mode == OUT_ACC) dst[i + e] += a[e];
                    else dst[i + e] = a[e];
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------
// Row-pass tile: 8192 consecutive floats = 4096 float2 units u; element e = 2u + half.
// Register arrangements (thread -> its 16 units):
//   A: u = t + 256 k             registers hold u bits 11..8  (e bits 12..9); coalesced
//   B: u = (t >> 4) << 8 | k << 4 | (t & 15)      registers hold u bits 7..4 (e bits 8..5)
//   C: u = t << 4 | k            registers hold u bits 3..0  (e bits 4..1): the thread
//                                owns the 32 consecutive coordinates 32 t .. 32 t + 31
// Shared memory holds unit u at u + 2 (u >> 4) (two pads per 16): conflict-free for the
// 64-bit accesses of arrangements A and B, and arrangement C's 16 consecutive units stay
// 16-byte aligned, so C moves them with eight 128-bit accesses.
// With a cluster (LC > 0) the 2^LC tiles of the cluster are consecutive in memory and the
// LC index bits above the tile are exchanged in the "slice" arrangement: register k holds
// unit rank * (4096 >> LC) + t + 256 * (k mod (16 >> LC)) of the tile of rank k / (16 >> LC).
// ---------------------------------------------------------------------------------
template <int ARR>
__device__ __forceinline__ int row_u(int t, int k)
{
    if (ARR == 0) return t + 256 * k;
    if (ARR == 1) return ((t >> 4) << 8) | (k << 4) | (t & 15);
    return (t << 4) | k;
}
__device__ __forceinline__ int row_pad(int u) { return u + 2 * (u >> 4); }
constexpr int kRowSmemUnits = 4096 + 512;

// row_pad(row_u<ARR>(t, k)) = row_base<ARR>(t) + kRowStride<ARR> * k: the part that depends
// on the thread is computed once, register k sits at a compile-time offset from it.
template <int ARR>
__device__ __forceinline__ int row_base(int t)
{
    if (ARR == 0) return t + 2 * (t >> 4);
    if (ARR == 1) return ((t >> 4) << 8) + ((t >> 4) << 5) + (t & 15);
    return 18 * t;
}
template <int ARR> struct RowStride { static constexpr int value = ARR == 0 ? 288 : ARR == 1 ? 18 : 1; };

template <int LC>
__device__ __forceinline__ int slice_u(int rank, int t, int k)
{
    return rank * (4096 >> LC) + t + 256 * (k & ((16 >> LC) - 1));
}

// Between arrangements B and C a unit moves only inside a group of 16 consecutive threads
// (unit t << 4 | k of arrangement C sits in thread (t & ~15) | k of arrangement B), so that
// exchange is ordered by a warp barrier; A <-> B crosses warps and takes the block barrier.
// A thread writes arrangement FROM at the addresses it read last in that arrangement, so
// back-to-back exchanges need no barrier between them.
template <int FROM, int TO>
__device__ __forceinline__ void row_exchange(u64 (&v)[16], u64* s)
{
    const int t = threadIdx.x;
    if (FROM == 2) {
        ulonglong2* p = reinterpret_cast<ulonglong2*>(s + row_base<2>(t));
#pragma unroll
        for (int k = 0; k < 8; ++k) p[k] = make_ulonglong2(v[2 * k], v[2 * k + 1]);
    } else {
        u64* p = s + row_base<FROM>(t);
#pragma unroll
        for (int k = 0; k < 16; ++k) p[RowStride<FROM>::value * k] = v[k];
    }
    if (FROM + TO == 3) __syncwarp();
    else __syncthreads();
    if (TO == 2) {
        const ulonglong2* p = reinterpret_cast<const ulonglong2*>(s + row_base<2>(t));
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const ulonglong2 w = p[k];
            v[2 * k] = w.x;
            v[2 * k + 1] = w.y;
        }
    } else {
        const u64* p = s + row_base<TO>(t);
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = p[RowStride<TO>::value * k];
    }
}

// butterflies over register index bits [B0, 4) of 16 packed units
template <int B0>
__device__ __forceinline__ void row_step(u64 (&v)[16])
{
#pragma unroll
    for (int b = B0; b < 4; ++b)
#pragma unroll
        for (int k = 0; k < 16; ++k)
            if (!(k & (1 << b))) bfly2(v[k], v[k | (1 << b)]);
}
__device__ __forceinline__ void row_step_inner(u64 (&v)[16])
{
#pragma unroll
    for (int k = 0; k < 16; ++k) v[k] = bfly_inner(v[k]);
}

// =================================================================================
// Sender, last pass: work -> low stages -> z = h/||y|| -> interval -> sum h Q(z) ->
// packed codes.  The thread ends with coordinates 32t..32t+31 of the tile and writes their
// W code words itself.
// =================================================================================
// Magnitude index of |z| in the 2^(W-1) positive intervals (Section 2.2.1): the number of
// positive boundaries strictly below |z|, found by arithmetic on the multiply-add pipe
// instead of compares and selects on the half-rate ALU pipe.
// With a boundary t held as T = -2^30 t, the saturated multiply-add sat(az 2^30 + T) is
// exactly 1 if az > t and exactly 0 otherwise: az - t is zero or at least one unit in the
// last place of t (2^-25 for the smallest boundary of the four-bit table, 2^-29 for that of
// the eight-bit one: the host checks that no boundary lies below 2^-7), which the factor
// 2^30 lifts to 1 or more, and the multiply-add rounds once.  The boundary of the next level is
// itself a multiply-add of that indicator (constants chosen on the host so that, rounded
// towards zero, it lands exactly on the fp32 boundary), and the index is the sum of the
// indicators (as a float 0..7) times the subnormal number 2^-149, whose bit pattern is the
// integer.  A NaN saturates to 0, so the index is always in range.
__device__ __forceinline__ float fma_sat(float a, float b, float c)
{
    float d;
    asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ u64 fma2_rz(u64 a, u64 b, u64 c)
{
    u64 r;
    asm("fma.rz.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ u64 mul2(u64 a, u64 b)
{
    u64 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// The constants of the search, those of the inner levels in both halves of a packed pair:
// two coordinates go through the tree together, their saturated multiply-adds one by one
// (no packed form saturates), everything else as one packed instruction for the two.
struct TreePairs {
    float big, k_root;
    u64 a1, b1, da, a_lo, db, b_lo, two, w1;
};
template <int W>
__device__ __forceinline__ TreePairs load_tree_pairs()
{
    const FmaTree& tr = c_tree[W];
    TreePairs tp;
    tp.big = tr.big;
    tp.k_root = tr.k_root;
    tp.a1 = pack2(tr.a1, tr.a1);
    tp.b1 = pack2(tr.b1, tr.b1);
    tp.da = pack2(tr.da, tr.da);
    tp.a_lo = pack2(tr.a_lo, tr.a_lo);
    tp.db = pack2(tr.db, tr.db);
    tp.b_lo = pack2(tr.b_lo, tr.b_lo);
    tp.two = pack2(2.f, 2.f);
    // W >= 4 takes the index times four, the byte offset of its value in the table; for
    // W >= 5 the tree of constants settles the top three bits of the index only
    const uint32_t unit = W >= 4 ? 4u << (W - 4) : 1u;
    tp.w1 = pack2(__uint_as_float(unit), __uint_as_float(unit));
    return tp;
}
// One coordinate through the same search with the constants taken straight from constant
// memory (no registers held): used where two tables are searched per coordinate
// (non-integer budgets).  Returns the index itself.
template <int W>
__device__ __forceinline__ uint32_t fma_magnitude_one(float az, const float* tbn)
{
    static_assert(W >= 1 && W <= 8, "code widths of the Lloyd-Max tables");
    if constexpr (W == 1) {
        return 0u;
    } else {
        const FmaTree& tr = c_tree[W];
        const float ir = fma_sat(az, tr.big, tr.k_root);
        float m = ir;
        if (W >= 3) {
            const float i1 = fma_sat(az, tr.big, __fmaf_rz(ir, tr.a1, tr.b1));
            m = fmaf(m, 2.f, i1);
            if (W >= 4) {
                const float t0 = __fmaf_rz(i1, __fmaf_rz(ir, tr.da, tr.a_lo), __fmaf_rz(ir, tr.db, tr.b_lo));
                m = fmaf(m, 2.f, fma_sat(az, tr.big, t0));
            }
        }
        // times a subnormal unit: the bit pattern is the integer (W >= 5: the byte offset of the octant)
        m *= __uint_as_float(W >= 5 ? 4u << (W - 4) : 1u);
        if constexpr (W >= 5) {
            const char* base = reinterpret_cast<const char*>(tbn);
#pragma unroll
            for (int step = 1 << (W - 5); step >= 1; step >>= 1) {
                const float b = *reinterpret_cast<const float*>(base + __float_as_uint(m) + 4 * (step - 1));
                m = fmaf(fma_sat(az, tr.big, b), __uint_as_float(4u * (uint32_t)step), m);
            }
            return __float_as_uint(m) >> 2;
        }
        return __float_as_uint(m);
    }
}

// `root`: the pair's indicators of the first level (for W = 2 they are the index itself)
// Returns the magnitude indices (W <= 3) or four times them, the byte offsets into a table
// of floats (W >= 4).  For W >= 5 the tree of constants finds the top three bits of the
// index (the seven boundaries at the eighth points of the table); the lower bits follow by
// bisection in `tbn`, the shared-memory table of the boundaries held as -2^30 t: one load,
// one saturated multiply-add and one (packed) multiply-add per level.
template <int W>
__device__ __forceinline__ void fma_magnitude_pair(float az0, float az1, const TreePairs& tp, uint32_t& m0, uint32_t& m1,
                                                   u64& root, const float* tbn = nullptr)
{
    static_assert(W >= 2 && W <= 8, "code widths of the Lloyd-Max tables");
    const u64 ir = pack2(fma_sat(az0, tp.big, tp.k_root), fma_sat(az1, tp.big, tp.k_root));
    root = ir;
    u64 m = ir;                                       // Horner form of 4 i_root + 2 i_1 + i_0
    if (W >= 3) {
        float t0, t1;
        unpack2(fma2_rz(ir, tp.a1, tp.b1), t0, t1);
        const u64 i1 = pack2(fma_sat(az0, tp.big, t0), fma_sat(az1, tp.big, t1));
        m = fma2(m, tp.two, i1);
        if (W >= 4) {
            unpack2(fma2_rz(i1, fma2_rz(ir, tp.da, tp.a_lo), fma2_rz(ir, tp.db, tp.b_lo)), t0, t1);
            const u64 i0 = pack2(fma_sat(az0, tp.big, t0), fma_sat(az1, tp.big, t1));
            m = fma2(m, tp.two, i0);
        }
    }
    float f0, f1;
    m = mul2(m, tp.w1);                               // times a subnormal unit: the bit pattern is the integer
    if constexpr (W >= 5) {
        const char* base = reinterpret_cast<const char*>(tbn);
#pragma unroll
        for (int step = 1 << (W - 5); step >= 1; step >>= 1) {
            unpack2(m, f0, f1);
            const float b0 = *reinterpret_cast<const float*>(base + __float_as_uint(f0) + 4 * (step - 1));
            const float b1 = *reinterpret_cast<const float*>(base + __float_as_uint(f1) + 4 * (step - 1));
            const u64 i = pack2(fma_sat(az0, tp.big, b0), fma_sat(az1, tp.big, b1));
            const float w = __uint_as_float(4u * (uint32_t)step);
            m = fma2(i, pack2(w, w), m);
        }
    }
    unpack2(m, f0, f1);
    m0 = __float_as_uint(f0);
    m1 = __float_as_uint(f1);
}

// The wide tables (W >= kCellMinWidth) in one step per coordinate (see c_cells): clamp, the
// cell's byte offset straight from the mantissa of |z| 2^(W+1) + 2^23 rounded towards zero
// (eight bytes per cell, three fraction bits masked off), one 64-bit load, one saturated
// multiply-add; the pair's indices (times four) by one packed multiply-add.
template <int W>
__device__ __forceinline__ void cell_magnitude_pair(float az0, float az1, const float2* cells, float zmax,
                                                    uint32_t& m0, uint32_t& m1)
{
    static_assert(W >= kCellMinWidth && W <= 8, "code widths with a cell table");
    constexpr float k8 = (float)(8 << (W - 2));
    static_assert(kCellMax * 8 <= 0x1000, "the offset mask below");
    const float c0 = fminf(az0, zmax), c1 = fminf(az1, zmax);
    const uint32_t o0 = __float_as_uint(__fmaf_rz(c0, k8, 8388608.f)) & 0xFF8u;
    const uint32_t o1 = __float_as_uint(__fmaf_rz(c1, k8, 8388608.f)) & 0xFF8u;
    const float2 e0 = *reinterpret_cast<const float2*>(reinterpret_cast<const char*>(cells) + o0);
    const float2 e1 = *reinterpret_cast<const float2*>(reinterpret_cast<const char*>(cells) + o1);
    const u64 ind = pack2(fma_sat(c0, 1073741824.f, e0.x), fma_sat(c1, 1073741824.f, e1.x));
    const float four = __uint_as_float(4u);                // subnormal: its bit pattern is the integer
    float f0, f1;
    unpack2(fma2(ind, pack2(four, four), pack2(e0.y, e1.y)), f0, f1);
    m0 = __float_as_uint(f0);
    m1 = __float_as_uint(f1);
}

// The thread's 32 consecutive coordinates -> their W words of the code bit stream
// (coordinate l in bits [l*W, l*W + W) of the 32*W-bit group), and sum |h| Q(|z|)
// (accumulated as sum |z| Q(|z|) for W > 1, so that |z| = |h| / ||y|| is formed once).
template <int W>
__device__ __forceinline__ void quantise_pack_32(const u64 (&v)[16], float inv_norm, bool live,
                                                 const float* s_tb, const float* s_tv, const float2* s_cells,
                                                 uint32_t (&words)[W], float& dot)
{
    [[maybe_unused]] const float zmax = c_cell_zmax[W];
    constexpr uint32_t half = 1u << (W - 1);
    if constexpr (W == 1) {
        // one bit per coordinate: the code is "not negative" and Q(|z|) is the same value
        // for every coordinate, so shift the sign bits in (coordinate 31 first) and sum |h|
        uint32_t negs = 0u;
        float sum = 0.f;
#pragma unroll
        for (int k = 15; k >= 0; --k) {
            float h0, h1;
            unpack2(v[k], h0, h1);
            negs = __funnelshift_l(__float_as_uint(h1), negs, 1);
            negs = __funnelshift_l(__float_as_uint(h0), negs, 1);
            sum += fabsf(h0) + fabsf(h1);
        }
        dot = sum * c_pos_value[0];
        words[0] = live ? ~negs : 0u;
    } else if constexpr (32 % W == 0) {
        // Widths that divide 32: a word holds 32 / W whole fields.  The fields collect the
        // magnitude indices (coordinates in descending order: shift the word up one field, drop
        // the index into the low bits); the top bit of every field (the code of a non-negative
        // coordinate is half + m) and the sign flips (a negative one has all W bits inverted)
        // are applied to the whole word at the end, the signs having been gathered by funnel shifts.
        constexpr int per = 32 / W;
        constexpr uint32_t lsb = W == 2 ? 0x55555555u : W == 4 ? 0x11111111u : 0x01010101u;
        static_assert(W == 2 || W == 4 || W == 8, "field widths that divide 32");
        const TreePairs tp = load_tree_pairs<W>();
        const u64 value_low2 = pack2(c_tree[2].v0, c_tree[2].v0), value_step2 = pack2(c_tree[2].dv, c_tree[2].dv);
        u64 dot2 = 0ull;
#pragma unroll
        for (int j = W - 1; j >= 0; --j) {
            // W = 4: the search returns 4 m (see load_tree_pairs), so the fields of a word are
            // collected times four, in two halves of four fields that cannot overflow
            uint32_t fields = 0u, fields_hi = 0u, signs = 0u;
#pragma unroll
            for (int i = per - 1; i >= 1; i -= 2) {
                const int l = j * per + i;                           // coordinates l (odd) and l - 1: one unit
                float h0, h1;
                unpack2(v[l >> 1], h0, h1);
                const float az0 = fabsf(h0) * inv_norm, az1 = fabsf(h1) * inv_norm;
                uint32_t m0, m1;
                float q0, q1;
                u64 root = 0ull;
                if constexpr (W >= kCellMinWidth) cell_magnitude_pair<W>(az0, az1, s_cells, zmax, m0, m1);
                else fma_magnitude_pair<W>(az0, az1, tp, m0, m1, root, s_tb);
                if constexpr (W == 2) {
                    // two values: the smaller plus the indicator times their distance (the sum may
                    // miss the larger value by one unit in the last place, far inside the scale's tolerance)
                    dot2 = fma2(pack2(az0, az1), fma2(root, value_step2, value_low2), dot2);
                } else {
                    q0 = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(s_tv) + m0);
                    q1 = *reinterpret_cast<const float*>(reinterpret_cast<const char*>(s_tv) + m1);
                    dot2 = fma2(pack2(az0, az1), pack2(q0, q1), dot2);
                    if constexpr (W == 8) {            // the fields take the index itself
                        m0 >>= 2;
                        m1 >>= 2;
                    }
                }
                // sums, not ORs: the compiler cannot know that an index fits its field
                if (W == 4 && i >= per / 2) fields_hi = (fields_hi * 16u + m1) * 16u + m0;
                else fields = ((((fields << W) + m1) << W) + m0);
                signs = __funnelshift_l(__float_as_uint(h1), signs, W);
                signs = __funnelshift_l(__float_as_uint(h0), signs, W);
            }
            if constexpr (W == 4) fields = (fields_hi << 14) + (fields >> 2);
            const uint32_t neg = (signs >> (W - 1)) & lsb;           // bit 0 of every field whose z is negative
            words[j] = live ? (fields | (lsb << (W - 1))) ^ ((neg << W) - neg) : 0u;
        }
        float d0, d1;
        unpack2(dot2, d0, d1);
        dot = d0 + d1;
    } else {
#pragma unroll
    for (int j = 0; j < W; ++j) words[j] = 0u;
    const TreePairs tp = load_tree_pairs<W>();
    // coordinates in descending order
#pragma unroll
    for (int k = 15; k >= 0; --k) {
        float h[2];
        unpack2(v[k], h[0], h[1]);
        const float az2[2] = {fabsf(h[0]) * inv_norm, fabsf(h[1]) * inv_norm};
        uint32_t m2[2];
        [[maybe_unused]] u64 root;
        if constexpr (W >= kCellMinWidth) cell_magnitude_pair<W>(az2[0], az2[1], s_cells, zmax, m2[0], m2[1]);
        else fma_magnitude_pair<W>(az2[0], az2[1], tp, m2[0], m2[1], root, s_tb);
#pragma unroll
        for (int e = 1; e >= 0; --e) {
            const int l = 2 * k + e;
            const float az = az2[e];
            uint32_t m = m2[e];
            if constexpr (W >= 4) {                    // the search returned the byte offset 4 m
                dot = fmaf(az, *reinterpret_cast<const float*>(reinterpret_cast<const char*>(s_tv) + m), dot);
                m >>= 2;
            } else {
                dot = fmaf(az, s_tv[m], dot);
            }
            // code = half + m for z >= 0 and half - 1 - m otherwise: set the top bit, then
            // flip all W bits where the sign bit of z (that of h) is set
            const uint32_t flip = (uint32_t)((int)__float_as_uint(h[e]) >> 31) & (2u * half - 1u);
            const uint32_t code = (m | half) ^ flip;
            const int a = (l * W) >> 5, off = (l * W) & 31;
            words[a] |= code << off;
            if (off + W > 32) words[a + 1] |= code >> (32 - off);
        }
    }
    if (!live) {
#pragma unroll
        for (int j = 0; j < W; ++j) words[j] = 0u;
    }
    }
    // wider codes summed |z| Q(|z|): back to the units of h (one division per thread and tile)
    if constexpr (W > 1) dot = live ? dot * __frcp_rn(inv_norm) : 0.f;
}

// ---------------------------------------------------------------------------------
// Non-integer budgets b > 1 (Section 4.1) on the row pass: the thread owns one group of 32
// coordinates; W = floor(b) + 1 words per group: (W-1)-bit fields, then one word whose bit l
// is the lowest code bit of coordinate l if its coin is set.
// ---------------------------------------------------------------------------------
// coins of the 32 coordinates of group g: two Philox calls of sixteen 8-bit numbers each.
// The four bytes of a word are compared with the threshold at once (one mask byte each) and
// the four answers gathered into a nibble by one multiplication.
__device__ __forceinline__ uint32_t group_coins(uint64_t seed, uint64_t g, uint32_t threshold)
{
    const uint32_t thr4 = threshold * 0x01010101u;
    uint32_t coins = 0u;
#pragma unroll
    for (int c = 0; c < 2; ++c) {
        const uint4 r = philox_stream(seed, 2u, 2 * g + c);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t lt = __vcmpltu4(w[j], thr4) & 0x01010101u;          // bit 8k: byte k is below the threshold
            // bits 0, 8, 16, 24 -> bits 28..31 (the partial products below bit 28 cannot carry into them)
            coins |= ((lt * 0x10204080u) >> 28) << (16 * c + 4 * j);
        }
    }
    return coins;
}

// tb_hi/tv_hi: positive boundaries (held as -2^30 t) and values of width W; tb_lo/tv_lo: of width W - 1
template <int W>
__device__ __forceinline__ void quantise_pack_frac(const u64 (&v)[16], float inv_norm, bool live, uint32_t coins,
                                                   const float* tb_hi, const float* tv_hi,
                                                   const float* tb_lo, const float* tv_lo,
                                                   uint32_t (&words)[W], float& dot)
{
    constexpr int W0 = W - 1;
    if constexpr (W == 2) {
        // 1 < b < 2 (the paper's own example is b = 1.5): one-bit codes, two-bit codes where the
        // coin is set.  The first word is the "not negative" bits either way (the upper bit of a
        // two-bit code is that bit too); the second holds index XOR sign of the coordinates with
        // a coin.  Signs and indices are gathered into words by funnel shifts and combined once
        // per thread; the value is c1 + coin * ((v0 - c1) + index * (v1 - v0)) by multiply-adds.
        const FmaTree& tr = c_tree[2];
        const float c1 = c_pos_value[0], lift = tr.v0 - c1;
        uint32_t negs = 0u, idx = 0u;
#pragma unroll
        for (int k = 15; k >= 0; --k) {
            float h[2];
            unpack2(v[k], h[0], h[1]);
#pragma unroll
            for (int e = 1; e >= 0; --e) {
                const int l = 2 * k + e;
                const float az = fabsf(h[e]) * inv_norm;
                const float ind = fma_sat(az, tr.big, tr.k_root);
                negs = __funnelshift_l(__float_as_uint(h[e]), negs, 1);
                idx = __funnelshift_l(__float_as_uint(fmaf(ind, -2.f, 0.5f)), idx, 1);     // its sign bit is the index
                const float coin = __uint_as_float((uint32_t)((int)(coins << (31 - l)) >> 31) & 0x3F800000u);
                dot = fmaf(az, fmaf(coin, fmaf(ind, tr.dv, lift), c1), dot);
            }
        }
        words[0] = live ? ~negs : 0u;
        words[1] = live ? (idx ^ negs) & coins : 0u;
        dot = live ? dot * __frcp_rn(inv_norm) : 0.f;
        return;
    }
#pragma unroll
    for (int j = 0; j < W; ++j) words[j] = 0u;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        float h[2];
        unpack2(v[k], h[0], h[1]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int l = 2 * k + e;
            const bool wide = (coins >> l) & 1u;
            const uint32_t hw = wide ? (1u << W0) : (1u << W0) >> 1;   // half the number of values
            const float az = fabsf(h[e]) * inv_norm;
            uint32_t m;
            if constexpr (W <= 3) {
                // both tables are searched (a few multiply-adds, no branches); the coin picks the result
                const uint32_t m_hi = fma_magnitude_one<W>(az, tb_hi), m_lo = fma_magnitude_one<W0>(az, tb_lo);
                m = wide ? m_hi : m_lo;
                dot = fmaf(az, wide ? tv_hi[m_hi] : tv_lo[m_lo], dot);
            } else {
                // one bisection in the coin's table (W0 levels for the wider table, the first of
                // them idle for the narrower one): a load, a saturated multiply-add and a
                // multiply-add per level, the index kept as a byte offset in a subnormal float
                const char* tb = reinterpret_cast<const char*>(wide ? tb_hi : tb_lo);
                const char* tv = reinterpret_cast<const char*>(wide ? tv_hi : tv_lo);
                const float big = c_tree[2].big;
                float mo = 0.f;
#pragma unroll
                for (int it = 0; it < W0; ++it) {
                    const int step = (1 << (W0 - 1)) >> it;
                    float ind = fma_sat(az, big, *reinterpret_cast<const float*>(tb + __float_as_uint(mo) + 4 * (step - 1)));
                    if (it == 0) ind = wide ? ind : 0.f;
                    mo = fmaf(ind, __uint_as_float(4u * (uint32_t)step), mo);
                }
                dot = fmaf(az, *reinterpret_cast<const float*>(tv + __float_as_uint(mo)), dot);
                m = __float_as_uint(mo) >> 2;
            }
            const uint32_t code = m ^ (__float_as_uint(h[e]) >> 31 ? hw - 1u : hw);
            const uint32_t field = wide ? code >> 1 : code;
            const int a = (l * W0) >> 5, off = (l * W0) & 31;
            words[a] |= field << off;
            if (off + W0 > 32) words[a + 1] |= field >> (32 - off);
            words[W0] |= (wide ? code & 1u : 0u) << l;          // bit l of the group's last word
        }
    }
    if (!live) {
#pragma unroll
        for (int j = 0; j < W; ++j) words[j] = 0u;
    }
    dot = live ? dot * __frcp_rn(inv_norm) : 0.f;      // summed as |z| Q(|z|): back to the units of h
}

// Uniform-interval family (Section 4.3) on the row pass: one signed byte per coordinate
// (the index n = round(z / delta), clamped to +-127), eight words per thread.
__device__ __forceinline__ void quantise_pack_uniform(const u64 (&v)[16], float inv_norm, bool live, float delta,
                                                      const float* s_tv, uint32_t (&words)[8], float& dot)
{
    const float inv_delta = __frcp_rn(delta);
#pragma unroll
    for (int j = 0; j < 8; ++j) words[j] = 0u;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        float h[2];
        unpack2(v[k], h[0], h[1]);
#pragma unroll
        for (int e = 0; e < 2; ++e) {
            const int l = 2 * k + e;
            const float z = h[e] * inv_norm;
            const int m = uniform_magnitude(fabsf(z), delta, inv_delta);
            dot = fmaf(fabsf(h[e]), s_tv[m], dot);
            // two's complement of +-m by the sign bit of z (m = 0 gives 0 for either sign),
            // its low byte moved into byte l % 4 of the word
            const int sgn = (int)__float_as_uint(z) >> 31;
            const uint32_t n = (uint32_t)((m ^ sgn) - sgn);
            const uint32_t sel = (l & 3) == 0 ? 0x3214u : (l & 3) == 1 ? 0x3240u : (l & 3) == 2 ? 0x3410u : 0x4210u;
            words[l >> 2] = __byte_perm(words[l >> 2], n, sel);
        }
    }
    if (!live) {
#pragma unroll
        for (int j = 0; j < 8; ++j) words[j] = 0u;
    }
}

// Shared-memory tables of the row pass of the sender: positive boundaries and values of
// width W, and of width W - 1 for non-integer budgets.
template <int W, bool FRAC>
struct EncTables {
    float tb[1 << (W - 1)], tv[1 << (W - 1)];
    float tb0[FRAC && W > 1 ? 1 << (W - 2) : 1], tv0[FRAC && W > 1 ? 1 << (W - 2) : 1];
    // one-step search of the wide tables (integer budgets): see c_cells
    float2 cells[!FRAC && W >= kCellMinWidth ? kCellMax : 1];
    // uniform-interval family (W = 8): the 128 values of this client by magnitude index
    __device__ __forceinline__ void fill_uniform(int t, const float* __restrict__ values)
    {
        for (int j = t; j < 128; j += kFastThreads) tv[j] = values[j];
    }
    __device__ __forceinline__ void fill(int t)
    {
        constexpr int half = 1 << (W - 1);
        // the searches work with saturated multiply-adds: boundaries are held as -2^30 t
        for (int j = t; j < half; j += kFastThreads) {
            tb[j] = -1073741824.f * c_pos_boundary[table_offset(W) + j];
            tv[j] = c_pos_value[table_offset(W) + j];
        }
        if constexpr (!FRAC && W >= kCellMinWidth)
            for (int j = t; j < c_cell_count[W]; j += kFastThreads) cells[j] = c_cells[W - kCellMinWidth][j];
        if (FRAC)
            for (int j = t; j < (half >> 1); j += kFastThreads) {
                tb0[j] = -1073741824.f * c_pos_boundary[table_offset(W > 1 ? W - 1 : 1) + j];
                tv0[j] = c_pos_value[table_offset(W > 1 ? W - 1 : 1) + j];
            }
    }
};

// The W code words of the thread's 32 coordinates, as one or two 128-bit stores where the
// width allows (code buffers are 16-byte aligned on this path).
template <int W>
__device__ __forceinline__ void store_words(uint32_t* dst, const uint32_t (&words)[W])
{
    if constexpr (W == 2) {
        *reinterpret_cast<uint2*>(dst) = make_uint2(words[0], words[1]);
    } else if constexpr (W == 4 || W == 8) {
#pragma unroll
        for (int j = 0; j < W; j += 4)
            *reinterpret_cast<uint4*>(dst + j) = make_uint4(words[j], words[j + 1], words[j + 2], words[j + 3]);
    } else {
#pragma unroll
        for (int j = 0; j < W; ++j) dst[j] = words[j];
    }
}

// The 13 stages of one tile held in arrangement A, then quantise, pack and store the tile's
// code words; returns the thread's part of sum |h| Q(|z|).
template <int W, bool FRAC, bool UNI = false>
// `norm2` points at the client's sum of squares; thread 0 turns it into 1/||y|| (0 for a
// zero or non-finite vector) in `s_inv`, which the block barrier of the first exchange
// publishes: one double-precision square root and division per tile instead of one per
// thread.  Where a middle pass ran before, it has left the value in `inv_ready` and the
// thread only copies it (the square root's latency would hold up that barrier).
// The caller makes sure that no thread still reads `s_inv` from an earlier tile.
__device__ __forceinline__ float enc_last_tile(u64 (&v)[16], const ClientDesc& cd, const double* norm2, uint64_t base,
                                               u64* s, const EncTables<W, FRAC>& tab, float* s_inv,
                                               const float* inv_ready = nullptr)
{
    const int t = threadIdx.x;
    if (t == 0) {
        if (W > 1 && inv_ready) {
            *s_inv = *inv_ready;
        } else {
            const double n2 = *norm2;
            const bool ok = n2 > 0.0 && n2 < INFINITY;
            if (W == 1) *s_inv = ok ? 1.f : 0.f;       // one-bit codes are the signs of h: only "live" matters
            else *s_inv = ok ? (float)(1.0 / sqrt(n2)) : 0.f;
        }
    }
    row_step<0>(v);                 // e bits 12..9
    row_exchange<0, 1>(v, s);
    row_step<0>(v);                 // e bits 8..5
    row_exchange<1, 2>(v, s);
    row_step<0>(v);                 // e bits 4..1
    row_step_inner(v);              // e bit 0
    const float inv_norm = *s_inv;
    const bool live = inv_norm > 0.f;
    uint32_t words[W];
    float dot = 0.f;
    if constexpr (UNI) {
        static_assert(W == 8 && !FRAC, "the uniform-interval family sends one byte per coordinate");
        quantise_pack_uniform(v, inv_norm, live, cd.delta, tab.tv, words, dot);
    } else if constexpr (FRAC && W >= 2) {
        const uint32_t coins = group_coins(cd.seed, (base >> 5) + t, cd.coin_thr);
        quantise_pack_frac<W>(v, inv_norm, live, coins, tab.tb, tab.tv, tab.tb0, tab.tv0, words, dot);
    } else {
        quantise_pack_32<W>(v, inv_norm, live, tab.tb, tab.tv, tab.cells, words, dot);
    }
    __builtin_assume(__isGlobal(cd.codes));
    store_words<W>(cd.codes + ((base >> 5) + t) * W, words);
    return dot;
}

// `work0`: the intermediate vector of the launch's first client; the clients' vectors follow
// one another 2^L floats apart, so a block's tile address needs no descriptor and its loads
// start at once.
template <int W, int LC, bool FRAC, bool UNI = false>
// Resident blocks per SM: five for one- and two-bit codes (48 registers, a few words spilled:
// 5580 -> 5870 GB/s at W = 1 against four); four from three bits on and for non-integer
// budgets, whose search constants and coins want the 64 registers (W = 4: 4140 GB/s with
// four blocks and no spills, 3960 with five and 68 bytes spilled).  Six run slower at every width.
__global__ void __launch_bounds__(kFastThreads, (FRAC || W >= 3 ? 4 : 5))
k_f_enc_last(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states, const float* __restrict__ work0, int L,
             int inv_ready, uint32_t tile0,
             float* __restrict__ scales /* small rounds: the block that finishes a client writes its scale S; else nullptr */,
             uint32_t* __restrict__ status)
{
    __shared__ __align__(16) u64 s[kRowSmemUnits];
    __shared__ float s_warp_dot[kFastThreads / 32];
    __shared__ float s_inv;
    __shared__ EncTables<W, FRAC> tab;
    const int t = threadIdx.x;
    const uint64_t base = (uint64_t)(blockIdx.x + tile0) << kFastTileLog;
    u64 v[16];
    if (LC == 0) {
        const u64* __restrict__ src = reinterpret_cast<const u64*>(work0 + ((uint64_t)blockIdx.y << L) + base);
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = src[row_u<0>(t, k)];
    }
    const ClientDesc cd = descs[blockIdx.y];
    if (UNI) tab.fill_uniform(t, cd.utable);
    else tab.fill(t);
    if (LC != 0) {
        // fetch this block's slice of all tiles of the cluster, do the stages across the
        // tiles, hand every result to the block that owns its tile
        cg::cluster_group cluster = cg::this_cluster();
        const int rank = (int)(blockIdx.x & ((1u << LC) - 1));
        const uint64_t base0 = (uint64_t)(blockIdx.x >> LC) << (kFastTileLog + LC);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int owner = k >> (4 - LC);
            v[k] = reinterpret_cast<const u64*>(cd.work + base0 + ((uint64_t)owner << kFastTileLog))
                       [slice_u<LC>(rank, t, k)];
        }
        row_step<4 - LC>(v);
        cluster_sync_execution();                      // every block of the cluster is running
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            u64* rs = cluster.map_shared_rank(s, k >> (4 - LC));
            rs[row_pad(slice_u<LC>(rank, t, k))] = v[k];
        }
        cluster_sync_publish();                        // the block's own tile is complete
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = s[row_pad(row_u<0>(t, k))];
        __syncthreads();                               // s is rewritten by the next exchange
    }
    const float dot = enc_last_tile<W, FRAC, UNI>(v, cd, &states[blockIdx.y].norm2, base, s, tab, &s_inv,
                                                  inv_ready ? &states[blockIdx.y].factor : nullptr);
    // the tile's 8192 terms are summed in fp32 (warp shuffles, then eight warp totals), which
    // is good to a few parts in 10^7; the tiles are summed in double
    float w = dot;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) w += __shfl_xor_sync(0xffffffffu, w, o);
    if ((t & 31) == 0) s_warp_dot[t >> 5] = w;
    __syncthreads();
    if (t == 0) {
        float tot = 0.f;
#pragma unroll
        for (int j = 0; j < kFastThreads / 32; ++j) tot += s_warp_dot[j];
        ClientState* st = &states[blockIdx.y];
        atomicAdd(&st->dot, (double)tot);
        if (scales) {
            // Small rounds save a launch: every tile counts itself in after its sum has gone out
            // (the fence orders the two), and the tile that counts last has all sums before it
            // and forms S = ||y||^2 sqrt(D) / sum h Q (Section 2.3) like k_enc_scale.  An
            // arrival counter, nobody waits.  (Large rounds keep the separate kernel: a fence
            // per tile costs them more than one launch.)
            __threadfence();
            if (atomicAdd(&st->tiles_done, 1u) == (1u << (L - kFastTileLog)) - 1u) {
                __threadfence();
                const double dot_all = atomicAdd(&st->dot, 0.0), n2 = st->norm2;
                uint32_t flags = 0;
                double S = 0.0;
                if (!(n2 < INFINITY)) flags |= 0x2u;
                else if (n2 == 0.0) flags |= 0x1u;
                else S = cd.extra_scale * n2 * sqrt((double)(1ull << L)) / dot_all;
                scales[cd.index] = (float)S;
                st->flags = flags;
                if (flags) atomicOr(status, flags);
            }
        }
    }
}

// ---------------------------------------------------------------------------------
// Sender, last pass, persistent form: a resident set of blocks walks all tiles of all
// clients of the launch (tile g belongs to client g >> tiles_log).  The next tile of a block
// is brought into a staging buffer in shared memory by one bulk asynchronous copy
// (cp.async.bulk, completion on an mbarrier) while the block works on the tile it holds in
// registers, so the global-memory latency of a tile is hidden behind the arithmetic of the
// one before it.  Every wait on the mbarrier is bounded; a wait that runs out raises
// EDEN_STATUS_TIMEOUT and the block returns after one more bounded wait for that copy.
// ---------------------------------------------------------------------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t arrivals)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// one arrival that announces `bytes` of asynchronous copies, then the copy itself
__device__ __forceinline__ void bulk_load_tile(void* dst_smem, const void* src_global, uint32_t bytes, uint64_t* bar)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_addr(dst_smem)), "l"(src_global), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}

// waits for the phase of the given parity; false if about two seconds pass first
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity)
{
    const long long t0 = clock64();
    for (;;) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\t"
                     "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                     "selp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(smem_addr(bar)), "r"(parity) : "memory");
        if (done) return true;
        if (clock64() - t0 > 4000000000ll) return false;
    }
}

constexpr uint32_t kStatusTimeout = 0x8u;   // EDEN_STATUS_TIMEOUT
constexpr uint32_t kStagedDynamicBytes = 4u << kFastTileLog;   // one tile

template <int W, bool FRAC>
__global__ void __launch_bounds__(kFastThreads, 3)
k_f_enc_last_staged(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states,
                    uint32_t total_tiles, int tiles_log, uint32_t* __restrict__ status)
{
    extern __shared__ __align__(128) unsigned char staged_dyn[];   // kStagedDynamicBytes: the staging buffer
    u64* stage = reinterpret_cast<u64*>(staged_dyn);
    __shared__ __align__(16) u64 s[kRowSmemUnits];
    __shared__ __align__(8) uint64_t bar;
    __shared__ double red[32];
    __shared__ int s_fail;
    __shared__ float s_inv;
    __shared__ EncTables<W, FRAC> tab;
    const int t = threadIdx.x;
    constexpr uint32_t kTileBytes = 4u << kFastTileLog;
    tab.fill(t);
    if (t == 0) {
        s_fail = 0;
        mbar_init(&bar, 1);
    }
    __syncthreads();
    uint32_t g = blockIdx.x;
    if (t == 0 && g < total_tiles) {
        const ClientDesc& c0 = descs[g >> tiles_log];
        bulk_load_tile(stage, c0.work + ((uint64_t)(g & ((1u << tiles_log) - 1u)) << kFastTileLog), kTileBytes, &bar);
    }
    uint32_t parity = 0;
    uint32_t cur = 0xFFFFFFFFu;          // client whose partial sum `acc` holds
    double acc = 0.0;
    for (; g < total_tiles; g += gridDim.x) {
        if (!mbar_wait_bounded(&bar, parity)) s_fail = 1;
        parity ^= 1u;
        u64 v[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = stage[row_u<0>(t, k)];
        __syncthreads();                               // the staging buffer is free again
        if (s_fail) break;
        const uint32_t gn = g + gridDim.x;
        if (t == 0 && gn < total_tiles) {
            const ClientDesc& cn = descs[gn >> tiles_log];
            bulk_load_tile(stage, cn.work + ((uint64_t)(gn & ((1u << tiles_log) - 1u)) << kFastTileLog), kTileBytes, &bar);
        }
        const uint32_t client = g >> tiles_log;
        if (client != cur) {
            if (cur != 0xFFFFFFFFu) {
                const double tot = block_sum(acc, red);
                if (t == 0) atomicAdd(&states[cur].dot, tot);
            }
            cur = client;
            acc = 0.0;
        }
        const ClientDesc cd = descs[client];
        const uint64_t base = (uint64_t)(g & ((1u << tiles_log) - 1u)) << kFastTileLog;
        acc += (double)enc_last_tile<W, FRAC>(v, cd, &states[client].norm2, base, s, tab, &s_inv);
        // the barrier after the next tile's staging read orders this tile's last exchange
        // reads before the next tile's first exchange writes
    }
    if (s_fail) {
        // the copy whose wait ran out may still be in flight and would land in shared memory
        // that the next block on this SM owns: give it one more bounded wait before leaving
        // (no further copy was started after the failure)
        mbar_wait_bounded(&bar, parity ^ 1u);
        if (t == 0) atomicOr(status, kStatusTimeout);
        return;
    }
    if (cur != 0xFFFFFFFFu) {
        const double tot = block_sum(acc, red);
        if (t == 0) atomicAdd(&states[cur].dot, tot);
    }
}

// =================================================================================
// Receiver, first pass: codes -> centroids (lost packets -> 0) -> low stages -> work
// =================================================================================
template <int W, int LC, bool FRAC>
__global__ void __launch_bounds__(kFastThreads, 4)
k_f_dec_first(const ClientDesc* __restrict__ descs, uint32_t tile0,
              ClientState* __restrict__ states /* small rounds: tile 0 of a client does k_dec_prep's work; else nullptr */,
              const float* __restrict__ scales, uint32_t* __restrict__ status)
{
    __shared__ __align__(16) u64 s[kRowSmemUnits];
    __shared__ float s_val[2 << W];                    // the 2^W values by code, then 2^W zeros
    __shared__ float s_val0[FRAC ? (1 << W) : 1];      // the same for width W - 1 (non-integer budgets)
    const ClientDesc cd = descs[blockIdx.y];
    const int t = threadIdx.x;
    constexpr int half = 1 << (W - 1);
    for (int j = t; j < (2 << W); j += kFastThreads) {
        float c = 0.f;
        if (j < (1 << W)) {
            if (W == 8 && cd.utable) c = uniform_byte_value((uint32_t)j, cd.utable);   // Section 4.3: the byte is the signed index
            else c = j >= half ? c_pos_value[table_offset(W) + j - half]
                               : -c_pos_value[table_offset(W) + half - 1 - j];
        }
        s_val[j] = c;
    }
    if (FRAC && W >= 2)
        for (int j = t; j < (1 << W); j += kFastThreads) {
            constexpr int h0 = half >> 1;
            float c = 0.f;
            if (j < (1 << (W - 1))) c = j >= h0 ? c_pos_value[table_offset(W > 1 ? W - 1 : 1) + j - h0]
                                                : -c_pos_value[table_offset(W > 1 ? W - 1 : 1) + h0 - 1 - j];
            s_val0[j] = c;
        }
    if (states && blockIdx.x + tile0 == 0u && t < 32) {
        // received fraction p and the factor S / (p sqrt D) of this client (Section 4.2), for
        // the last pass: one warp counts the bitmap (small rounds only: a few words)
        const uint64_t D = 1ull << cd.L;
        const uint64_t bits = (D + (1ull << cd.recv_shift) - 1) >> cd.recv_shift;
        uint32_t cnt = 0u;
        if (cd.recv) {
            for (uint64_t w = t; w < (bits + 31) >> 5; w += 32) {
                uint32_t word = cd.recv[w];
                const uint64_t left = bits - (w << 5);
                if (left < 32) word &= (1u << left) - 1u;
                cnt += (uint32_t)__popc(word);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
        }
        if (t == 0) {
            const double got = cd.recv ? (double)cnt : (double)bits;
            const double coords = D >= (1ull << cd.recv_shift) ? got * (double)(1ull << cd.recv_shift) : got * (double)D;
            const double p = coords / (double)D;
            ClientState* st = &states[blockIdx.y];
            const uint32_t flags = coords == 0.0 ? 0x4u : 0u;
            st->received = p;
            st->factor = flags ? 0.f : (float)((double)scales[cd.index] / (p * sqrt((double)D)) * cd.mean_scale);
            st->flags = flags;
            if (flags) atomicOr(status, flags);
        }
    }
    __syncthreads();
    const uint64_t base = (uint64_t)(blockIdx.x + tile0) << kFastTileLog;
    // the tile is 8 packets of 1024 coordinates; this thread's 32 coordinates lie in one.
    // A lost packet reads the zero half of the table (Section 4.2: lost coordinates are 0).
    const uint64_t pkt = (base >> 10) + (uint64_t)(t >> 5);
    const bool per_coord = W == 1 && cd.recv && cd.recv_shift == 0u;      // one bit per coordinate (W = 1 only)
    const bool arrived = cd.recv && !per_coord ? ((cd.recv[pkt >> 5] >> (pkt & 31)) & 1u) != 0u : true;
    const float* tbl = s_val + (arrived ? 0 : (1 << W));
    uint32_t words[W];
    const uint32_t* src = cd.codes + ((base >> 5) + t) * W;
    __builtin_assume(__isGlobal(src));
    __builtin_assume(__isGlobal(cd.work));
    // the thread's W words in one or two 128-bit (W = 2: 64-bit) loads where the message is
    // 16-byte aligned (the C ABI asks only for 4 bytes on this side)
    if ((W == 2 || W == 4 || W == 8) && (reinterpret_cast<uintptr_t>(cd.codes) & 15u) == 0) {
        if constexpr (W == 2) {
            const uint2 w2 = __ldg(reinterpret_cast<const uint2*>(src));
            words[0] = w2.x;
            words[W > 1 ? 1 : 0] = w2.y;
        } else {
#pragma unroll
            for (int j = 0; j + 3 < W; j += 4) {
                const uint4 w4 = __ldg(reinterpret_cast<const uint4*>(src + j));
                words[j] = w4.x;
                words[j + 1 < W ? j + 1 : 0] = w4.y;
                words[j + 2 < W ? j + 2 : 0] = w4.z;
                words[j + 3 < W ? j + 3 : 0] = w4.w;
            }
        }
    } else {
#pragma unroll
        for (int j = 0; j < W; ++j) words[j] = __ldg(src + j);
    }
    u64 v[16];
    if constexpr (FRAC && W >= 2) {
        // non-integer budget: (W-1)-bit fields, then the extra bits of the coordinates whose coin is set
        constexpr int W0 = W - 1;
        const uint32_t coins = group_coins(cd.seed, (base >> 5) + t, cd.coin_thr);
        // One load per coordinate, no branches: the shared-memory address of the value in the
        // wider table (field and extra bit) and in the narrower one (field alone) are both
        // formed, the coin's mask picks one.  Both include the offset of the zero half for
        // a lost packet.
        const uint32_t hi_addr = smem_addr(s_val) + (arrived ? 0u : (4u << W));
        const uint32_t lo_addr = smem_addr(s_val0) + (arrived ? 0u : (4u << W0));
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float q[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int l = 2 * k + e;
                const int a = (l * W0) >> 5, off = (l * W0) & 31;
                uint32_t x;                                     // the field at bits [2, W0 + 2): its byte offset
                if (off >= 2) x = off + W0 > 32 ? __funnelshift_r(words[a], words[a + 1 < W ? a + 1 : a], off - 2)
                                                : words[a] >> (off - 2);
                else x = words[a] << (2 - off);
                const uint32_t fb = x & (((1u << W0) - 1u) << 2);
                const uint32_t eb = (l >= 2 ? words[W0] >> (l - 2) : words[W0] << (2 - l)) & 4u;   // the extra bit, times four
                const uint32_t wide = (uint32_t)((int)(coins << (31 - l)) >> 31);                  // all ones if the coin is set
                const uint32_t addr = ((hi_addr + 2u * fb + eb) & wide) | ((lo_addr + fb) & ~wide);
                asm("ld.shared.f32 %0, [%1];" : "=f"(q[e]) : "r"(addr));
            }
            v[k] = pack2(q[0], q[1]);
        }
    } else if (W == 1) {
        // one bit per coordinate: +-c (or +-0 for a lost packet) by moving the bit into the sign
        const uint32_t minus_c = __float_as_uint(tbl[0]) | 0x80000000u;
        if (per_coord) {
            // the thread's 32 coordinates are one word of the bitmap: a coordinate that was not sent is 0
            const uint32_t kept = cd.recv[(base >> 5) + t];
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const uint32_t b0 = (words[0] << (31 - 2 * k)) & 0x80000000u;
                const uint32_t b1 = (words[0] << (30 - 2 * k)) & 0x80000000u;
                const uint32_t k0 = (uint32_t)((int)(kept << (31 - 2 * k)) >> 31);
                const uint32_t k1 = (uint32_t)((int)(kept << (30 - 2 * k)) >> 31);
                v[k] = pack2(__uint_as_float((minus_c ^ b0) & k0), __uint_as_float((minus_c ^ b1) & k1));
            }
        } else {
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const uint32_t b0 = (words[0] << (31 - 2 * k)) & 0x80000000u;
            const uint32_t b1 = (words[0] << (30 - 2 * k)) & 0x80000000u;
            v[k] = pack2(__uint_as_float(minus_c ^ b0), __uint_as_float(minus_c ^ b1));
        }
        }
    } else {
        // the field is moved straight to bits [2, W + 2) (one shift), masked and merged with
        // the bit that selects the zero half of the table (one logic operation): that is
        // the byte offset of the value, added to the table's address by the load itself
        const uint32_t lost = arrived ? 0u : (4u << W);
        const char* tbl_bytes = reinterpret_cast<const char*>(s_val);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            float q[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int l = 2 * k + e;
                const int a = (l * W) >> 5, off = (l * W) & 31;
                uint32_t x;
                if (off >= 2) x = off + W > 32 ? __funnelshift_r(words[a], words[a + 1 < W ? a + 1 : a], off - 2)
                                               : words[a] >> (off - 2);
                else x = words[a] << (2 - off);
                const uint32_t byte_off = (x & (((1u << W) - 1u) << 2)) | lost;
                q[e] = *reinterpret_cast<const float*>(tbl_bytes + byte_off);
            }
            v[k] = pack2(q[0], q[1]);
        }
    }
    row_step_inner(v);              // e bit 0
    row_step<0>(v);                 // e bits 4..1
    row_exchange<2, 1>(v, s);
    row_step<0>(v);                 // e bits 8..5
    row_exchange<1, 0>(v, s);
    row_step<0>(v);                 // e bits 12..9
    if (LC == 0) {
        u64* dst = reinterpret_cast<u64*>(cd.work + base);
#pragma unroll
        for (int k = 0; k < 16; ++k) dst[row_u<0>(t, k)] = v[k];
    } else {
        cg::cluster_group cluster = cg::this_cluster();
        const int rank = (int)(blockIdx.x & ((1u << LC) - 1));
        const uint64_t base0 = (uint64_t)(blockIdx.x >> LC) << (kFastTileLog + LC);
        __syncthreads();                               // readers of the last exchange are done
#pragma unroll
        for (int k = 0; k < 16; ++k) s[row_pad(row_u<0>(t, k))] = v[k];
        cluster_sync_publish();
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const u64* rs = cluster.map_shared_rank(s, k >> (4 - LC));
            v[k] = rs[row_pad(slice_u<LC>(rank, t, k))];
        }
        row_step<4 - LC>(v);                           // the LC stages across the tiles (consumes the fetched values)
        cluster_sync_execution();                      // nobody reads this block's tile any more
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int owner = k >> (4 - LC);
            reinterpret_cast<u64*>(cd.work + base0 + ((uint64_t)owner << kFastTileLog))
                [slice_u<LC>(rank, t, k)] = v[k];
        }
    }
}

}  // namespace eden
