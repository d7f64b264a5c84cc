// Device-side building blocks shared by the EDEN kernels: the Philox4x32-10 counter
// generator (shared randomness, EDEN Section 2.1), block reductions/scans and the
// descriptors the host hands to the kernels.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace eden {

// Per-client arguments of one call (host-built, copied to the device once per call).
struct ClientDesc {
    const float* src;        // encode: fp32 input row (x_c, or the compacted vector for b < 1)
    float* work;             // fp32[D] intermediate of the multi-pass transform
    uint32_t* codes;         // packed codes (encode writes, decode reads)
    const uint32_t* recv;    // decode: bitmap of what arrived (bit j = coordinates [j << recv_shift, (j + 1) << recv_shift)) or nullptr
    uint64_t seed;           // shared seed
    uint64_t valid;          // number of meaningful coordinates before padding (d or k)
    uint64_t d;              // input dimension
    uint32_t W;              // code width in bits
    uint32_t L;              // log2 of the rotation dimension D
    uint32_t subbit;         // 1 if b < 1
    uint32_t index;          // position of this client in the caller's arrays
    uint32_t coin_thr;       // non-integer b > 1: coin threshold round(frac * 256); else 0
    float delta;             // uniform-interval family (Section 4.3): interval width; else 0
    uint32_t recv_shift;     // log2 coordinates per bit of `recv`: 10 (packets), or 0 (one bit per coordinate, W = 1 only)
    uint32_t recv_ones;      // the number of set bits of `recv` where the caller knows it (a mask of exact size), else 0
    double extra_scale;      // encode: d/k for b < 1 (folded into S), else 1
    double mean_scale;       // decode: 1/n for the mean, 1 for accumulate
    const float* utable;     // uniform-interval family: values of magnitude index 0..127; else nullptr
};

// Per-client values produced on the device.
struct ClientState {
    double norm2;            // sum y_i^2
    double dot;              // sum h_i Q(z_i)
    double received;         // fraction of coordinates received
    float factor;            // decode: S / (p sqrt D) * mean_scale
    uint32_t flags;
    uint32_t tiles_done;     // encode, small rounds: tiles of the last pass that have added their part of `dot`
    uint32_t reserved;
};

// Result of the exact-size mask selection for one (seed, d, k): coordinate i is kept
// iff key_i < tau, or key_i == tau and it is among the first `rem` such coordinates.
struct MaskSelect {
    uint32_t bin_hi;         // top 16 bits of tau
    uint32_t below_hi;       // keys with top bits < bin_hi
    uint32_t tau;
    uint32_t rem;
    uint32_t below;          // keys < tau
    uint32_t fallback;       // one-pass selection: tau was outside the predicted band, redo with the histogram round
    uint32_t pad[2];
};

// ----------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of two 32x32->64
// multiplies with a Weyl key schedule.
// ----------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
        k.x += 0x9E3779B9u;
        k.y += 0xBB67AE85u;
    }
    return c;
}

__device__ __forceinline__ uint4 philox_stream(uint64_t seed, uint32_t stream, uint64_t call)
{
    return philox4x32_10(make_uint4((uint32_t)call, (uint32_t)(call >> 32), stream, 0u),
                         make_uint2((uint32_t)seed, (uint32_t)(seed >> 32)));
}

// The 32 sign bits (1 = minus) of rotated coordinates 32*g .. 32*g+31.
__device__ __forceinline__ uint32_t sign_word(uint64_t seed, uint64_t g)
{
    const uint4 r = philox_stream(seed, 0u, g >> 2);
    const uint32_t w = (uint32_t)g & 3u;
    return w == 0 ? r.x : w == 1 ? r.y : w == 2 ? r.z : r.w;
}

// Coin of rotated coordinate i for a non-integer budget b > 1 (Section 4.1: the
// coordinates that get the extra bit are picked by shared randomness): Philox stream 2,
// call i/16 yields sixteen 8-bit numbers, coordinate i takes number i%16 (the bytes of word
// 0 from the low one up, then word 1, ...); the coin is set iff the number is below the threshold.
__device__ __forceinline__ bool coin_bit(uint64_t seed, uint64_t i, uint32_t threshold)
{
    const uint4 r = philox_stream(seed, 2u, i >> 4);
    const uint32_t w = ((uint32_t)i >> 2) & 3u;
    const uint32_t word = w == 0 ? r.x : w == 1 ? r.y : w == 2 ? r.z : r.w;
    return ((word >> (8u * ((uint32_t)i & 3u))) & 0xFFu) < threshold;
}

// Uniform-interval family I_Delta (Section 4.3): magnitude index of |z| = the number of
// boundaries fl(delta * (k - 1/2)), k = 1..127, strictly below |z| (an endpoint belongs to
// the interval nearer zero; indices beyond 127 fall into the open outermost interval).
// The candidate floor(|z|/delta + 1/2 - 2^-10) is the index or one below it (the 2^-10
// outweighs every rounding error of the candidate's arithmetic, which stays below 4e-5 for
// quotients up to 127), so one comparison with the next boundary, formed exactly as
// defined, settles it.  The floor is taken by adding 2^23 with rounding towards minus
// infinity, which leaves the integer in the low mantissa bits and, as a float, in t - 2^23.
constexpr int kUniformMaxIndex = 127;
__device__ __forceinline__ int uniform_magnitude(float az, float delta, float inv_delta)
{
    const float u = fminf(fmaf(az, inv_delta, 0.5f - 0.0009765625f), (float)kUniformMaxIndex - 0.5f);
    const float t = __fadd_rd(u, 8388608.f);                   // 2^23 + floor(u), floor(u) in 0..126
    const float next = __fmul_rn(delta, t - 8388607.5f);       // boundary floor(u) + 1: delta * (floor(u) + 1/2)
    return (int)(__float_as_uint(t) & 0xFFu) + (az > next ? 1 : 0);
}
// value of a message byte: the byte is the signed index n, |n| <= 127 (-128 reads as -127)
__device__ __forceinline__ float uniform_byte_value(uint32_t byte, const float* values)
{
    const int n = (int)(int8_t)byte;
    const int m = min(n < 0 ? -n : n, kUniformMaxIndex);
    return n < 0 ? -values[m] : values[m];
}

// The four 32-bit mask keys of input coordinates 4t .. 4t+3.
__device__ __forceinline__ uint4 mask_keys(uint64_t seed, uint64_t t)
{
    return philox_stream(seed, 1u, t);
}

// ----------------------------------------------------------------------------------
// Block-wide helpers (blockDim.x a multiple of 32, at most 1024).
// ----------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Sum over the block; the result is valid in thread 0.  `scratch` holds 32 doubles.
__device__ __forceinline__ double block_sum(double v, double* scratch)
{
    v = warp_sum(v);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    double r = 0.0;
    if (warp == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        r = lane < nw ? scratch[lane] : 0.0;
        r = warp_sum(r);
    }
    __syncthreads();
    return r;
}

// Exclusive prefix sum of v over the block (thread order); *total gets the block sum.
// `scratch` holds 33 entries.
__device__ __forceinline__ unsigned long long block_exclusive_scan(unsigned long long v,
                                                                  unsigned long long* scratch,
                                                                  unsigned long long* total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        unsigned long long t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) scratch[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        const int nw = (blockDim.x + 31) >> 5;
        unsigned long long w = lane < nw ? scratch[lane] : 0ull;
        unsigned long long winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            unsigned long long t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        scratch[lane] = winc - w;            // exclusive offset of each warp
        if (lane == 31) scratch[32] = winc;  // block total
    }
    __syncthreads();
    const unsigned long long r = scratch[warp] + inc - v;
    *total = scratch[32];
    __syncthreads();
    return r;
}

}  // namespace eden
