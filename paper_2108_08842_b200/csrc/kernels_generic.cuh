// Shape-generic transform kernels: any rotation dimension, any pass split.  A tile of
// 2^lt floats is staged in shared memory and a range of its index bits is transformed
// with radix-8 register butterflies between barriers.  These kernels serve the small and
// odd shapes; the register-blocked kernels in kernels_fast.cuh take over the large
// power-of-two shapes.
//
// Tile geometry (PassGeom): a tile is 2^lr rows of 2^lw consecutive coordinates, the rows
// 2^lo coordinates apart.  With lr = 0 and lw = lo = lt it is a contiguous run (a "row
// pass" over index bits [0, lt)); otherwise the pass transforms the row bits
// [lo, lo + lr) of the global index (a "column pass").
#pragma once
#include "eden_device.cuh"

namespace eden {

struct PassGeom {
    int lt;   // log2 of the tile size
    int lw;   // log2 of the contiguous run
    int lo;   // log2 of the distance between rows
    int lr;   // log2 of the number of rows
};

constexpr int kGenericThreads = 256;
constexpr int kGenericTileLog = 13;                      // largest generic tile: 8192 floats
constexpr int kGenericPerThread = (1 << kGenericTileLog) / kGenericThreads;

__device__ __forceinline__ uint64_t tile_coord(const PassGeom& g, uint64_t tile, int e)
{
    const int chunk_bits = g.lo - g.lw;
    const uint64_t outer = tile >> chunk_bits;
    const uint64_t chunk = tile & ((1ull << chunk_bits) - 1);
    const uint64_t r = (uint64_t)(e >> g.lw);
    const uint64_t c = (uint64_t)(e & ((1 << g.lw) - 1));
    return (outer << (g.lo + g.lr)) + (r << g.lo) + (chunk << g.lw) + c;
}

// Walsh-Hadamard butterflies over index bits [b0, b1) of a shared-memory tile of 2^lt
// floats: pair (a, b) -> (a + b, a - b), up to three bits per barrier.
__device__ __forceinline__ void tile_fwht(float* s, int lt, int b0, int b1)
{
    for (int sh = b0; sh < b1; sh += 3) {
        const int nb = min(3, b1 - sh);
        const int groups = (1 << lt) >> nb;
        for (int gi = threadIdx.x; gi < groups; gi += blockDim.x) {
            const int lo = gi & ((1 << sh) - 1);
            const int e0 = ((gi >> sh) << (sh + nb)) | lo;
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k < (1 << nb)) v[k] = s[e0 + (k << sh)];
#pragma unroll
            for (int b = 0; b < 3; ++b) {
                if (b < nb) {
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        if (!(k & (1 << b)) && (k | (1 << b)) < (1 << nb)) {
                            const float a = v[k], c = v[k | (1 << b)];
                            v[k] = a + c;
                            v[k | (1 << b)] = a - c;
                        }
                    }
                }
            }
#pragma unroll
            for (int k = 0; k < 8; ++k)
                if (k < (1 << nb)) s[e0 + (k << sh)] = v[k];
        }
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------
// Quantiser tables in constant memory: for each width W the 2^(W-1) - 1 positive
// interval boundaries and the 2^(W-1) positive values (Section 3).  Widths 1..8 are
// laid out one after the other: width W starts at offset 2^(W-1) - 1 in both arrays
// (the boundary array of width W has one unused slot at its end).
// ---------------------------------------------------------------------------------
__constant__ float c_pos_boundary[256];
__constant__ float c_pos_value[256];

__device__ __forceinline__ int table_offset(int W) { return (1 << (W - 1)) - 1; }

// The interval search of Section 2.2.1 as arithmetic on the multiply-add pipe (see
// fma_magnitude_pair in kernels_fast.cuh); for code widths above 4 the tree covers the
// seven boundaries at the eighth points of the table.  A boundary t is held as
// -2^30 t; `a*`/`d*` are differences of such values, chosen on the host so that the
// multiply-adds below (rounded towards zero) land exactly on the fp32 boundaries.
struct FmaTree {
    float big;                   // 2^30
    float k_root;                // the root of the search tree
    float a1, b1;                // second level (W >= 3):  fma(i_root, a1, b1)
    float a_lo, da, b_lo, db;    // third level (W = 4):     fma(i_2, fma(i_root, da, a_lo), fma(i_root, db, b_lo))
    float v0, dv;                // W = 2: the smaller positive value and the step to the larger
    float pad[6];
};
__constant__ FmaTree c_tree[9];  // by code width

// The same search for the wide tables (W >= kCellMinWidth) in one step: the positive axis is
// cut into cells of width 2^-(W-2), narrower than the smallest gap between two boundaries of
// the table, so that a cell holds at most one boundary; floor(|z| 2^(W-2)) picks the cell,
// whose entry gives that boundary (as -2^30 t; a cell without one holds -3e38, which never
// fires) and the number of boundaries below the cell, and one saturated multiply-add decides
// the boundary inside.  Entry: x = -2^30 t, y = the float whose bit pattern is four times
// the count (the byte offset of a value in a table of floats).  The last cell lies wholly
// above the last boundary, and |z| is clamped to its middle (c_cell_zmax).
constexpr int kCellMinWidth = 5;
constexpr int kCellMax = 288;
__constant__ float2 c_cells[9 - kCellMinWidth][kCellMax];
__constant__ float c_cell_zmax[9];
__constant__ int c_cell_count[9];

// Interval rule of Section 2.2.1 on one normalised coordinate: magnitude index m =
// number of positive boundaries strictly below |z| (an endpoint belongs to the interval
// nearer zero), by a branch-free binary search over the sorted boundaries in `tb`.
__device__ __forceinline__ int magnitude_index(float az, const float* tb, int half)
{
    int m = 0;
    for (int step = half >> 1; step >= 1; step >>= 1)
        m += (az > tb[m + step - 1]) ? step : 0;
    return m;
}

// =================================================================================
// Sender
// =================================================================================

// First pass of a multi-pass encode (a column pass over the top bits): reads the input
// (zero beyond `valid`), flips signs (Diag(s), Section 5), accumulates ||y||^2 and writes
// the partially transformed tile to the work buffer.
__global__ void __launch_bounds__(kGenericThreads)
k_enc_first(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states, PassGeom g)
{
    extern __shared__ float s[];
    __shared__ double red[32];
    const ClientDesc cd = descs[blockIdx.y];
    const int T = 1 << g.lt;
    float local = 0.f;
    for (int e = threadIdx.x; e < T; e += blockDim.x) {
        const uint64_t i = tile_coord(g, blockIdx.x, e);
        float v = i < cd.valid ? cd.src[i] : 0.f;
        local = fmaf(v, v, local);
        const uint32_t sw = sign_word(cd.seed, i >> 5);
        if ((sw >> (i & 31)) & 1u) v = -v;
        s[e] = v;
    }
    __syncthreads();
    tile_fwht(s, g.lt, g.lw, g.lw + g.lr);
    for (int e = threadIdx.x; e < T; e += blockDim.x)
        cd.work[tile_coord(g, blockIdx.x, e)] = s[e];
    const double tot = block_sum((double)local, red);
    if (threadIdx.x == 0) atomicAdd(&states[blockIdx.y].norm2, tot);
}

// Middle pass, in place on the work buffer (used by sender and receiver).
__global__ void __launch_bounds__(kGenericThreads)
k_mid(const ClientDesc* __restrict__ descs, PassGeom g)
{
    extern __shared__ float s[];
    const ClientDesc cd = descs[blockIdx.y];
    const int T = 1 << g.lt;
    for (int e = threadIdx.x; e < T; e += blockDim.x) s[e] = cd.work[tile_coord(g, blockIdx.x, e)];
    __syncthreads();
    tile_fwht(s, g.lt, g.lw, g.lw + g.lr);
    for (int e = threadIdx.x; e < T; e += blockDim.x) cd.work[tile_coord(g, blockIdx.x, e)] = s[e];
}

// Last pass of the encode (a row pass over the low bits): finishes the transform,
// normalises (z = h / ||y||, i.e. eta_x R(x) of Section 2.2.1), finds each coordinate's
// interval, accumulates sum h_i Q(z_i) for the scale (Section 2.3) and writes the packed
// codes (a bit stream of W-bit fields, assembled with warp-wide OR reductions).  SINGLE: the whole vector is one tile, so this kernel
// also loads the input, flips the signs and computes the norm.
template <bool SINGLE>
__global__ void __launch_bounds__(kGenericThreads)
k_enc_last(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states, PassGeom g)
{
    extern __shared__ float s[];
    __shared__ double red[32];
    __shared__ double s_norm2;
    __shared__ float s_tb[128], s_tv[128];     // table of width W
    __shared__ float s_tb0[64], s_tv0[64];     // table of width W - 1 (non-integer budgets)
    const ClientDesc cd = descs[blockIdx.y];
    const int T = 1 << g.lt;
    const int W = (int)cd.W, half = 1 << (W - 1);
    const bool frac = cd.coin_thr != 0u;       // then W = floor(b) + 1
    const int Wf = frac ? W - 1 : W;           // width of the fixed fields
    const bool uniform = cd.utable != nullptr;  // Section 4.3: W = 8, the byte is the signed index
    for (int j = threadIdx.x; j < half; j += blockDim.x) {
        s_tb[j] = c_pos_boundary[table_offset(W) + j];
        s_tv[j] = uniform ? cd.utable[j] : c_pos_value[table_offset(W) + j];
    }
    if (frac)
        for (int j = threadIdx.x; j < (half >> 1); j += blockDim.x) {
            s_tb0[j] = c_pos_boundary[table_offset(W - 1) + j];
            s_tv0[j] = c_pos_value[table_offset(W - 1) + j];
        }
    const uint64_t base = (uint64_t)blockIdx.x << g.lt;
    if (SINGLE) {
        float local = 0.f;
        for (int e = threadIdx.x; e < T; e += blockDim.x) {
            const uint64_t i = base + e;
            float v = i < cd.valid ? cd.src[i] : 0.f;
            local = fmaf(v, v, local);
            const uint32_t sw = sign_word(cd.seed, i >> 5);
            if ((sw >> (i & 31)) & 1u) v = -v;
            s[e] = v;
        }
        const double tot = block_sum((double)local, red);
        if (threadIdx.x == 0) { s_norm2 = tot; states[blockIdx.y].norm2 = tot; }
    } else {
        for (int e = threadIdx.x; e < T; e += blockDim.x) s[e] = cd.work[base + e];
        if (threadIdx.x == 0) s_norm2 = states[blockIdx.y].norm2;
    }
    __syncthreads();
    tile_fwht(s, g.lt, 0, g.lt);
    const double n2 = s_norm2;
    const bool live = n2 > 0.0 && n2 < INFINITY;
    const float inv_norm = live ? (float)(1.0 / sqrt(n2)) : 0.f;
    const int lane = threadIdx.x & 31;
    float dot = 0.f;
    const float inv_delta = uniform ? __frcp_rn(cd.delta) : 0.f;
    const int Tr = (T + 31) & ~31;                     // whole warps take part in the reductions
    const uint64_t D = (uint64_t)1 << cd.L;
    const uint64_t total_words = frac ? ((D + 31) >> 5) * W : (D * W + 31) >> 5;
    for (int e = threadIdx.x; e < Tr; e += blockDim.x) {
        const float h = e < T ? s[e] : 0.f;
        const float z = h * inv_norm;
        // non-integer budget: this coordinate uses the wider table iff its coin is set
        const bool coin = frac && e < T && coin_bit(cd.seed, base + e, cd.coin_thr);
        const bool wide = !frac || coin;
        const int hw = wide ? half : half >> 1;
        const float* tb = wide ? s_tb : s_tb0;
        const float* tv = wide ? s_tv : s_tv0;
        const int m = uniform ? uniform_magnitude(fabsf(z), cd.delta, inv_delta) : magnitude_index(fabsf(z), tb, hw);
        const bool neg = z < 0.f;
        uint32_t code = neg ? (uint32_t)(hw - 1 - m) : (uint32_t)(hw + m);
        if (uniform) code = (uint32_t)(neg ? -m : m) & 0xFFu;
        const float q = neg ? -tv[m] : tv[m];
        if (e < T) dot = fmaf(h, q, dot); else code = 0u;
        if (!live) code = 0u;
        // the 32 lanes hold 32 consecutive Wf-bit fields = Wf words of the bit stream:
        // lane l's field starts at bit l*Wf of the group
        const uint32_t field = coin ? code >> 1 : code;
        uint32_t mine = 0u;
        for (int j = 0; j < Wf; ++j) {
            const int sh = lane * Wf - 32 * j;
            uint32_t part = 0u;
            if (sh > -Wf && sh < 32) part = sh >= 0 ? field << sh : field >> (-sh);
            const uint32_t word = __reduce_or_sync(0xffffffffu, part);
            if (lane == j) mine = word;
        }
        if (frac) {
            // last word of the group: bit l = lowest code bit of coordinate l if its coin is set
            const uint32_t word = __ballot_sync(0xffffffffu, coin && (code & 1u));
            if (lane == Wf) mine = word;
        }
        const uint64_t widx = ((base + e) >> 5) * W + lane;
        if (lane < W && widx < total_words) cd.codes[widx] = mine;
    }
    const double tot = block_sum((double)dot, red);
    if (threadIdx.x == 0) {
        if (SINGLE) states[blockIdx.y].dot = tot;
        else atomicAdd(&states[blockIdx.y].dot, tot);
    }
}

// S_c = ||y||^2 / <R(y), Q> = ||y||^2 sqrt(D) / sum h_i Q(z_i), times d/k below one bit.
__global__ void k_enc_scale(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states,
                            float* __restrict__ scales, uint32_t n,
                            uint32_t* __restrict__ status)
{
    const uint32_t c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= n) return;
    const ClientDesc cd = descs[c];
    ClientState st = states[c];
    uint32_t flags = 0;
    double S = 0.0;
    if (!(st.norm2 < INFINITY)) flags |= 0x2u;             // inf or nan
    else if (st.norm2 == 0.0) flags |= 0x1u;
    else S = cd.extra_scale * st.norm2 * sqrt((double)(1ull << cd.L)) / st.dot;
    scales[cd.index] = (float)S;
    states[c].flags = flags;
    if (flags) atomicOr(status, flags);
}

// =================================================================================
// Receiver
// =================================================================================

// Per client: received fraction p (Section 4.2) and the factor S / (p sqrt D) that the
// last pass applies (times 1/n for the mean).  One block per client.
__global__ void __launch_bounds__(256)
k_dec_prep(const ClientDesc* __restrict__ descs, ClientState* __restrict__ states,
           const float* __restrict__ scales, uint32_t* __restrict__ status)
{
    __shared__ double red[32];
    const ClientDesc cd = descs[blockIdx.x];
    const uint64_t D = 1ull << cd.L;
    const uint64_t per_bit = 1ull << cd.recv_shift;                  // coordinates per bit of the bitmap
    const uint64_t packets = (D + per_bit - 1) >> cd.recv_shift;
    double cnt = 0.0;
    if (cd.recv && cd.recv_ones) {
        if (threadIdx.x == 0) cnt = (double)cd.recv_ones;            // a mask of known size: nothing to count
    } else if (cd.recv) {
        const uint64_t words = (packets + 31) >> 5;
        // eight loads in flight per thread: a bitmap with one bit per coordinate (the mask of the
        // other order of Section 4.1) is megabytes long and one block walks it
        uint32_t ones = 0u;
        for (uint64_t w0 = threadIdx.x; w0 < words; w0 += 8ull * blockDim.x) {
            uint32_t v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const uint64_t w = w0 + (uint64_t)u * blockDim.x;
                v[u] = w < words ? cd.recv[w] : 0u;
                const uint64_t left = w < words ? packets - (w << 5) : 32;
                if (left < 32) v[u] &= (1u << left) - 1u;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) ones += (uint32_t)__popc(v[u]);
            if (ones >= 0x80000000u) {                      // keep the 32-bit partial count from wrapping
                cnt += (double)ones;
                ones = 0u;
            }
        }
        cnt += (double)ones;
    } else if (threadIdx.x == 0) {
        cnt = (double)packets;
    }
    const double tot = block_sum(cnt, red);
    if (threadIdx.x == 0) {
        const double coords = D >= per_bit ? tot * (double)per_bit : tot * (double)D;
        const double p = coords / (double)D;
        uint32_t flags = 0;
        float f = 0.f;
        if (coords == 0.0) flags = 0x4u;
        else f = (float)((double)scales[cd.index] / (p * sqrt((double)D)) * cd.mean_scale);
        states[blockIdx.x].received = p;
        states[blockIdx.x].factor = f;
        states[blockIdx.x].flags = flags;
        if (flags) atomicOr(status, flags);
    }
}

// Value of coordinate i of the received message: centroid of its code, 0 if its packet
// was lost (Section 4.2).  Called by all 32 lanes of a warp with 32 consecutive
// coordinates (lane = i % 32); `valid` is false for lanes beyond the vector.  `tv` holds
// the positive values of width W, `tv0` those of width W - 1 (non-integer budgets only).
__device__ __forceinline__ float received_value(const ClientDesc& cd, uint64_t i, bool valid,
                                                const float* tv, const float* tv0)
{
    const int W = (int)cd.W;
    const bool frac = cd.coin_thr != 0u;
    const bool coin = frac && valid && coin_bit(cd.seed, i, cd.coin_thr);
    if (!valid) return 0.f;
    if (cd.recv) {
        const uint64_t pkt = i >> cd.recv_shift;
        if (!((cd.recv[pkt >> 5] >> (pkt & 31)) & 1u)) return 0.f;
    }
    if (!frac) {
        const int half = 1 << (W - 1);
        const uint64_t bit = i * W;                        // field i of the bit stream
        const uint32_t off = (uint32_t)(bit & 31);
        uint32_t code = cd.codes[bit >> 5] >> off;
        if (off + W > 32) code |= cd.codes[(bit >> 5) + 1] << (32 - off);
        code &= (1u << W) - 1u;
        if (cd.utable) return uniform_byte_value(code, tv);
        return code >= (uint32_t)half ? tv[code - half] : -tv[half - 1 - code];
    }
    // non-integer budget: groups of 32 coordinates, W words each: (W-1)-bit fields, then one
    // word whose bit l is the extra bit of coordinate l (if its coin is set)
    const int W0 = W - 1;
    const uint32_t l = (uint32_t)(i & 31);
    const uint32_t* grp = cd.codes + (i >> 5) * W;
    const uint32_t bit = l * W0, off = bit & 31;
    uint32_t field = grp[bit >> 5] >> off;
    if (off + W0 > 32) field |= grp[(bit >> 5) + 1] << (32 - off);
    field &= (1u << W0) - 1u;
    if (coin) {
        const uint32_t code = (field << 1) | ((grp[W0] >> l) & 1u);
        const int half = 1 << (W - 1);
        return code >= (uint32_t)half ? tv[code - half] : -tv[half - 1 - code];
    }
    const int half0 = 1 << (W0 - 1);
    return field >= (uint32_t)half0 ? tv0[field - half0] : -tv0[half0 - 1 - field];
}

// OUT_PART: block row y sums its own run of the group's clients into partial vector y (the
// partial vectors are added up by k_sum_partials): more blocks when a round has few tiles.
enum OutMode { OUT_WRITE = 0, OUT_ACC = 1, OUT_YHAT = 2, OUT_PART = 3 };

// First pass of the decode (a row pass over the low bits): unpack, centroid lookup,
// lost packets to zero, low stages; writes the work buffer.
__global__ void __launch_bounds__(kGenericThreads)
k_dec_first(const ClientDesc* __restrict__ descs, PassGeom g)
{
    extern __shared__ float s[];
    __shared__ float s_tv[128], s_tv0[64];
    const ClientDesc cd = descs[blockIdx.y];
    const int T = 1 << g.lt;
    const int half = 1 << (cd.W - 1);
    for (int j = threadIdx.x; j < half; j += blockDim.x)
        s_tv[j] = cd.utable ? cd.utable[j] : c_pos_value[table_offset(cd.W) + j];
    if (cd.coin_thr)
        for (int j = threadIdx.x; j < (half >> 1); j += blockDim.x)
            s_tv0[j] = c_pos_value[table_offset(cd.W - 1) + j];
    __syncthreads();
    const uint64_t base = (uint64_t)blockIdx.x << g.lt;
    // T is a multiple of 32 here (multi-pass vectors), so whole warps call received_value
    for (int e = threadIdx.x; e < T; e += blockDim.x) s[e] = received_value(cd, base + e, true, s_tv, s_tv0);
    __syncthreads();
    tile_fwht(s, g.lt, 0, g.lt);
    for (int e = threadIdx.x; e < T; e += blockDim.x) cd.work[base + e] = s[e];
}

// Last pass of the decode: for each client of the group finish the inverse transform of
// this tile, apply the client's signs and factor (x_hat = (S/p) Diag(s) H q / sqrt D,
// Sections 2.2.2 and 4.2) and add it to a running sum kept in registers; the tile of the
// sum is written once.  FROM_CODES: the whole vector is one tile and the kernel starts
// from the packed codes.  OUT_YHAT stores one client's estimate of the compacted vector
// (b < 1) for the scatter kernel.
template <bool FROM_CODES>
__global__ void __launch_bounds__(kGenericThreads)
k_dec_last(const ClientDesc* __restrict__ descs_in, const ClientState* __restrict__ states_in,
           uint32_t n_group, PassGeom g, float* __restrict__ out, uint64_t d, int mode,
           uint32_t n_members, uint64_t part_stride)
{
    // OUT_YHAT: block row y handles member y alone (n_group = 1); OUT_PART: block row y sums
    // members [y * n_group, min((y + 1) * n_group, n_members)) into out + y * part_stride
    const uint32_t first = mode == OUT_YHAT ? blockIdx.y : mode == OUT_PART ? blockIdx.y * n_group : 0u;
    if (mode == OUT_PART) n_group = min(n_group, n_members - first);
    const ClientDesc* __restrict__ descs = descs_in + first;
    const ClientState* __restrict__ states = states_in + first;
    extern __shared__ float s[];
    __shared__ float s_tv[128], s_tv0[64];
    const int T = 1 << g.lt;
    float acc[kGenericPerThread];
#pragma unroll
    for (int k = 0; k < kGenericPerThread; ++k) acc[k] = 0.f;
    for (uint32_t c = 0; c < n_group; ++c) {
        const ClientDesc cd = descs[c];
        const float f = states[c].factor;
        if (FROM_CODES) {
            const int half = 1 << (cd.W - 1);
            __syncthreads();
            for (int j = threadIdx.x; j < half; j += blockDim.x)
                s_tv[j] = cd.utable ? cd.utable[j] : c_pos_value[table_offset(cd.W) + j];
            if (cd.coin_thr)
                for (int j = threadIdx.x; j < (half >> 1); j += blockDim.x)
                    s_tv0[j] = c_pos_value[table_offset(cd.W - 1) + j];
            __syncthreads();
            const int Tr = (T + 31) & ~31;               // whole warps call received_value
            for (int e = threadIdx.x; e < Tr; e += blockDim.x) {
                // FROM_CODES tiles are contiguous: coordinate = tile * T + e
                const float v = received_value(cd, ((uint64_t)blockIdx.x << g.lt) + e, e < T, s_tv, s_tv0);
                if (e < T) s[e] = v;
            }
        } else {
            for (int e = threadIdx.x; e < T; e += blockDim.x)
                s[e] = cd.work[tile_coord(g, blockIdx.x, e)];
        }
        __syncthreads();
        if (FROM_CODES) tile_fwht(s, g.lt, 0, g.lt);
        else tile_fwht(s, g.lt, g.lw, g.lw + g.lr);
#pragma unroll
        for (int k = 0; k < kGenericPerThread; ++k) {
            const int e = threadIdx.x + k * kGenericThreads;
            if (e < T) {
                const uint64_t i = tile_coord(g, blockIdx.x, e);
                const uint32_t sw = sign_word(cd.seed, i >> 5);
                const float v = s[e] * f;
                acc[k] += ((sw >> (i & 31)) & 1u) ? -v : v;
            }
        }
        __syncthreads();
    }
    const uint64_t limit = mode == OUT_YHAT ? (1ull << descs[0].L) : d;
    float* dst = mode == OUT_YHAT ? descs[0].work : mode == OUT_PART ? out + blockIdx.y * part_stride : out;
#pragma unroll
    for (int k = 0; k < kGenericPerThread; ++k) {
        const int e = threadIdx.x + k * kGenericThreads;
        if (e < T) {
            const uint64_t i = tile_coord(g, blockIdx.x, e);
            if (i < limit) {
                if (mode == OUT_ACC) dst[i] += acc[k];
                else dst[i] = acc[k];
            }
        }
    }
}

// out[i] (+)= sum over the G partial vectors of part[g * stride + i], i < d.
__global__ void __launch_bounds__(256)
k_sum_partials(const float* __restrict__ part, uint32_t G, uint64_t stride, uint64_t d,
               float* __restrict__ out, int accumulate)
{
    const uint64_t q = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;      // group of four coordinates
    const uint64_t i = q * 4;
    if (i >= d) return;
    if (i + 3 < d && (((uintptr_t)out) & 15u) == 0) {
        float4 a = accumulate ? *reinterpret_cast<const float4*>(out + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        for (uint32_t g = 0; g < G; ++g) {
            const float4 v = *reinterpret_cast<const float4*>(part + g * stride + i);
            a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w;
        }
        *reinterpret_cast<float4*>(out + i) = a;
    } else {
        for (uint64_t j = i; j < d && j < i + 4; ++j) {
            float a = accumulate ? out[j] : 0.f;
            for (uint32_t g = 0; g < G; ++g) a += part[g * stride + j];
            out[j] = a;
        }
    }
}

// =================================================================================
// Uniform-interval family (Section 4.3): occurrences of each index value in a client's
// message (D signed bytes), for the entropy coder's model and the coded-length estimate.
// hist[client][n + 128] counts index n.  Per-warp histograms in shared memory, flushed once.
// =================================================================================
constexpr int kHistThreads = 256;
constexpr int kHistBytesPerThread = 64;

__global__ void __launch_bounds__(kHistThreads)
k_index_hist(const int8_t* const* __restrict__ index, uint64_t D, uint32_t* __restrict__ hist)
{
    __shared__ uint32_t s_h[kHistThreads / 32][256];
    const int t = threadIdx.x, warp = t >> 5;
    for (int j = t; j < (kHistThreads / 32) * 256; j += kHistThreads) (&s_h[0][0])[j] = 0u;
    __syncthreads();
    const int8_t* __restrict__ src = index[blockIdx.y];
    const uint64_t units = D >> 4;                              // 16-byte units
    const uint64_t per_block = (uint64_t)kHistThreads * (kHistBytesPerThread / 16);
    for (uint64_t u0 = (uint64_t)blockIdx.x * per_block; u0 < units; u0 += (uint64_t)gridDim.x * per_block) {
#pragma unroll
        for (int r = 0; r < kHistBytesPerThread / 16; ++r) {
            const uint64_t u = u0 + (uint64_t)r * kHistThreads + t;
            if (u < units) {
                const uint4 w = reinterpret_cast<const uint4*>(src)[u];
                const uint32_t words[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b)
                        atomicAdd(&s_h[warp][(((words[a] >> (8 * b)) & 0xFFu) + 128u) & 0xFFu], 1u);
            }
        }
    }
    if (blockIdx.x == 0 && t < (int)(D & 15u))                  // D < 16: a few single bytes
        atomicAdd(&s_h[0][((uint32_t)(uint8_t)src[(units << 4) + t] + 128u) & 0xFFu], 1u);
    __syncthreads();
    uint32_t total = 0u;
#pragma unroll
    for (int w = 0; w < kHistThreads / 32; ++w) total += s_h[w][t];
    if (total) atomicAdd(&hist[(uint64_t)blockIdx.y * 256u + t], total);
}

}  // namespace eden
