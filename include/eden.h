/*
 * eden.h -- C ABI of the EDEN hot path on one NVIDIA B200 (sm_100a).
 *
 * EDEN (arXiv 2108.08842) estimates the mean of n client vectors x_c in R^d from one
 * short message per client.  This library implements the sender's compress step and
 * the receiver's decompress-and-average step (the paper's Figure 1) as CUDA kernels.
 *
 * Conventions shared by every entry point
 *   - "dev" pointers are CUDA device pointers on the context's device, "host" pointers
 *     are ordinary host memory.  The caller owns every buffer it passes in; the library
 *     owns nothing but the context object and never frees or reallocates caller memory.
 *   - Work is enqueued on the context's stream and is asynchronous unless stated.
 *     Host arrays (bits, seeds, pointer tables) are consumed before the call returns.
 *   - Every function returns EDEN_OK (0) or a negative EDEN_ERR_* code.  Nothing
 *     throws or aborts across this boundary.  Data-dependent conditions (a zero or
 *     non-finite vector, a client with no packet) are reported through the device
 *     status word, read with eden_status().
 *   - bits (the per-client budget b) and seed (the randomness a sender shares with the
 *     receiver, Section 2.1) are side information both sides agree on (Section 4.1
 *     leaves it to the two sides to transmit b or fix it beforehand); they are
 *     arguments on both sides and are not stored in the message.  Seeds must differ between clients and
 *     between rounds; that is the caller's duty.
 *   - Supported budgets: 0 < b <= 1 (one-bit codes; b < 1 adds the shared-seed
 *     sparsification of Section 4.1), the integers 2..8 (Section 3) and non-integer
 *     1 < b < 8 (Section 4.1: each coordinate is coded with 2^(floor(b)+1) values if its
 *     shared coin is set, with 2^floor(b) otherwise; coins are Philox stream 2, call t
 *     giving sixteen 8-bit numbers (the bytes of its four words, low byte first) for
 *     coordinates 16t..16t+15, set iff the number is below round((b - floor(b)) * 256),
 *     so the share of wider codes is a multiple of 1/256).  Other values return
 *     EDEN_ERR_UNSUPPORTED_BITS.
 *   - Rotation (Section 5): R = (1/sqrt D) H_D Diag(s), H_D the Sylvester-ordered
 *     Walsh-Hadamard matrix, D = 2^ceil(log2 d') with d' = d for b >= 1 and d' = the
 *     kept count k for b < 1; shorter vectors are zero-padded, all D coordinates are
 *     coded and the estimate is truncated back.  Signs s come from Philox4x32-10,
 *     key = seed, counter = (t, 0, stream, 0): stream 0 call t gives the 128 sign bits
 *     of coordinates 128t..128t+127 (word (i/32)%4, bit i%32, 1 = minus); stream 1
 *     call t gives the 32-bit mask keys of input coordinates 4t..4t+3.
 *   - Message layout: the codes form one little-endian bit stream of W-bit fields (W the
 *     code width): coordinate i occupies stream bits [i*W, i*W + W), low bit of the code
 *     first; stream bit b is bit b%32 of 32-bit word b/32.  A code is the rank of its
 *     quantisation value in ascending order.  A packet is 1024 consecutive rotated
 *     coordinates = 128*W bytes.  The scale S travels beside the codes as one fp32.
 *     Non-integer b: groups of 32 coordinates of W = floor(b)+1 words each: first the bit
 *     stream of floor(b)-bit fields (an unset coordinate's code, or the upper bits of a
 *     set coordinate's code), then one word whose bit l is the lowest code bit of the
 *     group's coordinate l if its coin is set, else 0.  Only floor(b)*32 + (coins set) bits
 *     of a group carry information (both sides know the coins); whole words keep packets
 *     at 128*W bytes.
 */
#ifndef EDEN_H_
#define EDEN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define EDEN_OK                    0
#define EDEN_ERR_INVALID_ARG      -1
#define EDEN_ERR_UNSUPPORTED_BITS -2
#define EDEN_ERR_CUDA             -3
#define EDEN_ERR_WORKSPACE        -4   /* workspace too small for this call */
#define EDEN_ERR_TOO_LARGE        -5   /* d beyond EDEN_MAX_DIM */

/* bits of the device status word (eden_status) */
#define EDEN_STATUS_ZERO_VECTOR  0x1u  /* some client had ||x|| = 0: scale 0, codes 0   */
#define EDEN_STATUS_NONFINITE    0x2u  /* some client's norm was inf/nan: its output is unspecified */
#define EDEN_STATUS_NO_DATA      0x4u  /* some client had no packet received: it was skipped */
#define EDEN_STATUS_TIMEOUT      0x8u  /* a bounded wait inside a kernel ran out: the call's output is unspecified */
#define EDEN_STATUS_SCRATCH      0x10u /* a b < 1 mask selection outgrew its candidate list (sized for a margin of
                                          twelve standard deviations): that client's mask, and so its output, is unspecified */

#define EDEN_PACKET_COORDS 1024u
#define EDEN_MAX_DIM       (1ull << 30)

typedef struct eden_ctx eden_ctx;

/* Per-client figures of the most recent eden_encode / eden_mean / eden_decode_accumulate
 * call (eden_client_stats). */
typedef struct eden_client_stat {
    double norm2;      /* encode: ||y||^2 of the (sparsified) vector that was rotated      */
    double dot;        /* encode: sum_i h_i Q(z_i) with h = H_D Diag(s) y (unnormalised)    */
    double received;   /* decode: fraction p of rotated coordinates that arrived           */
    uint32_t flags;    /* EDEN_STATUS_* bits that apply to this client                     */
    uint32_t reserved;
} eden_client_stat;

/* ---- size rules: pure host functions of (d, bits); no GPU work ------------------- */

/* k = d for bits >= 1, else floor(d*bits + 0.5) clamped to [1, d] (Section 4.1: the
 * mask has exactly d*p ones). */
uint64_t eden_kept_count(uint64_t d, double bits);
/* D = smallest power of two >= (bits >= 1 ? d : k)  (Section 5; zero padding). */
uint64_t eden_rot_dim(uint64_t d, double bits);
/* Widest code of a client: 1 for bits <= 1, bits for integer bits, floor(bits)+1 for
 * non-integer bits > 1; 0 if the budget is unsupported (Sections 3, 4.1). */
uint32_t eden_code_width(double bits);
/* bytes of one client's packed codes: ceil(D*W/32) words rounded up to a multiple of 16 bytes
 * (Section 2.2.1: ceil(log2 |I|) * d bits). */
uint64_t eden_code_bytes(uint64_t d, double bits);
/* ceil(D / 1024): packets of one client's message (Section 4.2). */
uint64_t eden_num_packets(uint64_t d, double bits);
/* 32-bit words of a received-packet bitmap: ceil(packets / 32). */
uint64_t eden_recv_mask_words(uint64_t d, double bits);
/* Bytes of device workspace that lets eden_encode / eden_mean process n_batch clients
 * of dimension up to d_max per launch group (any budgets).  A smaller workspace is
 * accepted as long as it holds one client: calls then run in several groups. */
uint64_t eden_workspace_bytes(uint64_t d_max, uint32_t n_batch);

/* The sweeps over HBM that one client's rotation (Section 5) takes for (d, bits) on the
 * default kernels, sender order: pass_bits[0..*n_passes) = index bits each sweep
 * transforms (they add up to log2 D); the last entry is the sweep that reads or writes
 * the codes.  Host only; pass_bits holds max_passes entries. */
int eden_pass_plan(uint64_t d, double bits, uint32_t* pass_bits, uint32_t max_passes,
                   uint32_t* n_passes);

/* The quantiser the library uses for code width W (1..8): 2^W values in ascending
 * order and the 2^W - 1 interval boundaries between them, rounded to fp32
 * (Section 3: Lloyd-Max for N(0,1), centre-of-mass values).  Host arrays, host only. */
int eden_table(uint32_t W, float* centroids, float* boundaries);

/* Host only.  The kernels search the intervals of code widths 2..4 with multiply-adds whose
 * constants are derived from the table above, and those of widths 5..8 through a table of
 * cells of width 2^-(W-2); EDEN_OK if every boundary that search can form is bit-identical
 * to the table's fp32 boundary, no boundary is too small for the kernels' exact
 * comparison, and no cell holds two boundaries (all hold for the tables of Section 3;
 * eden_create refuses to run otherwise). */
int eden_self_check(void);

/* ---- context ---------------------------------------------------------------------- */

/* Creates a context bound to a device, a stream (cudaStream_t passed as void*, NULL =
 * the default stream) and a caller-allocated device workspace (256-byte aligned).  The
 * context keeps pointers into the workspace; the caller must keep it alive and must
 * not use it while a call is in flight.  Uploads the quantiser tables (synchronous). */
int eden_create(eden_ctx** out, int cuda_device, void* cuda_stream,
                void* workspace_dev, uint64_t workspace_bytes);
int eden_destroy(eden_ctx* ctx);

/* ---- sender: Sections 2.2.1, 2.3, 4.1 --------------------------------------------- */

/* Compresses n independent clients.
 *   x      dev, fp32, n rows, row c starts at x + c*ld_x, ld_x >= d; read only.
 *   bits   host, n budgets.          seeds  host, n shared seeds.
 *   codes  host array of n dev pointers, each to eden_code_bytes(d, bits[c]) bytes,
 *          16-byte aligned; overwritten with the packed codes Q(eta_x R(x)).
 *   scales dev, fp32[n]; scales[c] = S_c = ||x_c||^2 / <R(x_c), Q(eta R(x_c))>
 *          (for b < 1: the scale of the sparsified, 1/p-rescaled vector).
 * A zero vector gives scale 0 and all-zero codes (status ZERO_VECTOR). */
int eden_encode(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                const double* bits, const uint64_t* seeds,
                uint8_t* const* codes, float* scales);

/* ---- receiver: Sections 2.2.2, 4.1, 4.2 ------------------------------------------- */

/* acc[i] += sum_c x_hat_c[i] over the n given clients, x_hat_c = (S_c/p_c) R_c^-1(Q_c)
 * scattered back through the client's sparsification mask when b < 1.
 *   codes      host array of n dev pointers (layout above); scales dev fp32[n].
 *   recv_masks host array of n dev pointers or NULL; entry c (NULL = nothing lost)
 *              points to eden_recv_mask_words() words, bit i of word i/32 = packet i
 *              arrived.  Lost coordinates count as 0 and p_c = received/D (Section 4.2).
 *   acc        dev fp32[d], read and written; 4-byte alignment is enough, a vector that
 *              is also 16-byte aligned takes the faster kernels (the same holds for the
 *              output of eden_mean and eden_mean_partial).
 *   n_used     host, optional: n is ADDED to *n_used (the caller zeroes it before the
 *              first call of a round and divides acc by it after the last); clients
 *              with no packet received are skipped and flagged (status NO_DATA) but
 *              still counted, because the mean of Section 2.2.2 is over all n senders.
 * No per-client estimate is stored for b >= 1; clients with b < 1 use the workspace. */
int eden_decode_accumulate(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                           const double* bits, const uint64_t* seeds,
                           const uint32_t* const* recv_masks,
                           uint64_t d, uint32_t n, float* acc, uint32_t* n_used);

/* mean[i] = (1/n) sum_c x_hat_c[i]; same inputs; mean (dev fp32[d]) is overwritten. */
int eden_mean(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
              const double* bits, const uint64_t* seeds,
              const uint32_t* const* recv_masks,
              uint64_t d, uint32_t n, float* mean);

/* This GPU's share of the mean when the n_total senders of a round are split over several
 * GPUs (the senders are independent until the final sum, Section 2.2.2):
 *     partial[i] = (1/n_total) sum over the n given clients of x_hat_c[i]     (overwritten)
 * so that the element-wise sum of the partial vectors of all GPUs (one all-reduce of d
 * floats, done by the caller) is the mean over all n_total senders.  n <= n_total. */
int eden_mean_partial(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                      const double* bits, const uint64_t* seeds,
                      const uint32_t* const* recv_masks,
                      uint64_t d, uint32_t n, uint64_t n_total, float* partial);

/* The sparsification mask of Section 4.1 for (seed, d, bits < 1) as a bitmap:
 * mask_bits dev, ceil(d/32) words, bit i of word i/32 = coordinate i is kept. */
int eden_sparsification_mask(eden_ctx* ctx, uint64_t seed, uint64_t d, double bits,
                             uint32_t* mask_bits);

/* The same mask as eden_sparsification_mask, for callers that cannot allocate device
 * memory and therefore have no workspace to build a context on: code running inside a
 * host application whose own allocator already holds the whole card, a service that
 * fixes its memory map at start-up, a loop that cannot afford the device-wide stall of
 * an allocation.  (The paper has no counterpart: this entry point exists for those
 * callers only.)  It needs no eden_ctx and calls no cudaMalloc/cudaFree or any other
 * allocating routine: its scratch (selection state, two 65536-bin histograms, per-chunk
 * counts; about 0.65 MB) is a fixed array inside the library, resident on every GPU that
 * loads the library until the process exits.
 *   cuda_device, cuda_stream   where to run (stream as void*, NULL = default stream)
 *   seed, d, bits              as for eden_sparsification_mask; 0 < bits < 1
 *   mask_bits                  dev, ceil(d/32) words, caller-owned, overwritten
 * Limits and rules: d <= EDEN_NOALLOC_MAX_DIM, larger d returns EDEN_ERR_TOO_LARGE.  The
 * first call on a device looks up the array's device address (once per device, with that
 * device made current); make that first call before any stream capture begins.  All
 * calls on a device share the one array, which keeps the previous call's contents (the
 * entry point clears what must start at zero): two calls whose GPU work overlaps -- two
 * streams, two threads -- race on it; run them on one stream or order them yourself.
 * Asynchronous on cuda_stream like the other entry points.  The calling thread's current
 * device is the same after the call as before it. */
#define EDEN_NOALLOC_MAX_DIM (1ull << 24)
int eden_sparsification_mask_noalloc(int cuda_device, void* cuda_stream, uint64_t seed,
                                     uint64_t d, double bits, uint32_t* mask_bits);

/* ---- Section 4.1, the other order: sparsification after the rotation ---------------- */

/* Section 4.1 notes that the random mask of a budget b < 1 can be applied before or after
 * the rotation, with about the same error; eden_encode applies it before (it shrinks the
 * transform).  These entry points apply it after: the sender rotates and codes the whole
 * vector with one bit per coordinate exactly as for b = 1 (same scale S) and sends only the
 * codes of a random mask over the D = eden_rot_dim(d, 1) ROTATED coordinates, exactly
 * k' = eden_after_kept_count(d, b) = floor(D b + 1/2) of them (at least 1): the k' smallest
 * (key, index) pairs of the seed's mask keys, indexed by rotated coordinate.  The message is
 * the kept codes in increasing index order, one bit each (bit j of the stream = code of the
 * j-th kept coordinate), eden_after_code_bytes(d, b) bytes, plus S.  The receiver rebuilds
 * the mask, takes it as the pattern of what arrived, puts 0 elsewhere and multiplies by
 * 1/p, p = k'/D: the receiver of Section 4.2 (Lemma 4.3) with this mask.  0 < b < 1 for
 * every client; D up to about 10^8 (larger returns EDEN_ERR_TOO_LARGE); no packet loss on
 * top.  The workspace must hold eden_after_workspace_bytes(d, n). */
uint64_t eden_after_kept_count(uint64_t d, double bits);
uint64_t eden_after_code_bytes(uint64_t d, double bits);
uint64_t eden_after_workspace_bytes(uint64_t d, uint32_t n);
/* codes: host array of n dev pointers, each eden_after_code_bytes(d, bits[c]) bytes, 16-byte
 * aligned, overwritten; other arguments as for eden_encode. */
int eden_encode_sparsify_after(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                               const double* bits, const uint64_t* seeds,
                               uint8_t* const* codes, float* scales);
/* mean[i] = (1/n) sum_c x_hat_c[i] (overwritten) / acc[i] += sum_c x_hat_c[i], *n_used += n;
 * codes 4-byte aligned; other arguments as for eden_mean / eden_decode_accumulate. */
int eden_mean_sparsify_after(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                             const double* bits, const uint64_t* seeds,
                             uint64_t d, uint32_t n, float* mean);
int eden_decode_accumulate_sparsify_after(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                                          const double* bits, const uint64_t* seeds,
                                          uint64_t d, uint32_t n, float* acc, uint32_t* n_used);

/* ---- Section 4.3: the uniform-interval family --------------------------------------- */

/* Section 4.3 replaces the 2^b Lloyd-Max intervals by
 *     I_Delta = { [Delta (n - 1/2), Delta (n + 1/2)] : n integer },
 * Delta_b = the smallest Delta whose entropy under N(0,1) is at most b bits, so that an
 * entropy coder (not part of this library) can send the indices in about b bits per
 * coordinate.  The interval of a coordinate is n = round(z / Delta) (an endpoint goes to
 * the interval nearer zero), its value the interval's centre of mass.  This library
 * clamps n to +-EDEN_UNIFORM_MAX_INDEX (the two outermost intervals run to infinity) and
 * writes one signed byte per rotated coordinate: byte i of a client's message is the
 * index of rotated coordinate i; a packet is still 1024 coordinates.  Supported widths:
 * EDEN_UNIFORM_MIN_DELTA <= Delta < 2 (Section 4.3 requires Delta in (0, 2)); other
 * values return EDEN_ERR_UNSUPPORTED_BITS.  No sparsification: budgets below
 * eden_uniform_entropy(2) ~ 1.24 bits are not reachable with this family. */
#define EDEN_UNIFORM_MAX_INDEX 127
#define EDEN_UNIFORM_MIN_DELTA 0.0625

/* Host only.  Entropy in bits per coordinate of I_Delta under N(0,1); 0 for delta <= 0. */
double eden_uniform_entropy(double delta);
/* Host only.  Delta_b for a budget of `bits` per coordinate; 0 if it falls outside the
 * supported widths. */
double eden_uniform_delta(double bits);
/* Host only.  values[m], m = 0..127: centre of mass of the interval of magnitude index m,
 * rounded to fp32 (what the kernels use); the value of index -m is -values[m]. */
int eden_uniform_values(double delta, float* values);
/* Bytes of one client's index message: the rotation dimension, rounded up to 16. */
uint64_t eden_uniform_index_bytes(uint64_t d);

/* eden_encode with Q over I_Delta.  delta: host, n interval widths.  index: host array
 * of n dev pointers, each to eden_uniform_index_bytes(d) bytes, 16-byte aligned.
 * scales as for eden_encode.  Same error and status behaviour. */
int eden_encode_uniform(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                        const double* delta, const uint64_t* seeds,
                        int8_t* const* index, float* scales);
/* eden_decode_accumulate / eden_mean for such messages (index pointers 4-byte aligned). */
int eden_decode_accumulate_uniform(eden_ctx* ctx, const int8_t* const* index, const float* scales,
                                   const double* delta, const uint64_t* seeds,
                                   const uint32_t* const* recv_masks,
                                   uint64_t d, uint32_t n, float* acc, uint32_t* n_used);
int eden_mean_uniform(eden_ctx* ctx, const int8_t* const* index, const float* scales,
                      const double* delta, const uint64_t* seeds,
                      const uint32_t* const* recv_masks,
                      uint64_t d, uint32_t n, float* mean);
/* Occurrences of each index value in each client's message: hist (dev, n * 256 words,
 * overwritten), hist[c * 256 + v + 128] = number of rotated coordinates of client c with
 * index v.  The empirical entropy of these counts estimates the entropy-coded length
 * (Section 4.3 and its appendix on representation length).  index pointers 16-byte
 * aligned. */
int eden_index_histogram(eden_ctx* ctx, const int8_t* const* index, uint64_t d, uint32_t n,
                         uint32_t* hist);

/* ---- the same two steps on host memory (copies included) --------------------------- */

/* x, codes (array of n host pointers), scales are HOST buffers (pinned memory makes the
 * copies asynchronous).  Copies x to the device, encodes, copies codes and scales back
 * and synchronises the stream.  Needs eden_host_workspace_bytes() of workspace.  Inputs
 * of 64 MiB and more are processed in chunks of clients on two internal side streams so
 * that uploads, kernels and downloads overlap; eden_client_stats then describes the last
 * chunk only. */
int eden_encode_host(eden_ctx* ctx, const float* x_host, uint64_t ld_x, uint64_t d, uint32_t n,
                     const double* bits, const uint64_t* seeds,
                     uint8_t* const* codes_host, float* scales_host);
/* codes, scales, recv_masks (entries may be NULL), mean are HOST buffers. */
int eden_mean_host(eden_ctx* ctx, const uint8_t* const* codes_host, const float* scales_host,
                   const double* bits, const uint64_t* seeds,
                   const uint32_t* const* recv_masks_host,
                   uint64_t d, uint32_t n, float* mean_host);
/* workspace for the two calls above: staging for n vectors, their codes and the mean
 * on top of eden_workspace_bytes(d, n). */
uint64_t eden_host_workspace_bytes(uint64_t d, uint32_t n);

/* ---- status ----------------------------------------------------------------------- */

/* Synchronises the stream and returns the OR of EDEN_STATUS_* bits raised since the
 * last eden_status call (then clears them). */
int eden_status(eden_ctx* ctx, uint32_t* device_status_word);
/* Synchronises and copies the per-client figures of the most recent call (host array, n). */
int eden_client_stats(eden_ctx* ctx, uint32_t n, eden_client_stat* out);
/* Number of kernels the library has launched on this context so far. */
uint64_t eden_launch_count(const eden_ctx* ctx);

/* Cross-checking aid: with on != 0 every call on this context uses the shape-generic
 * kernels instead of the register-blocked ones (same results, slower). */
int eden_force_generic_kernels(eden_ctx* ctx, int on);

/* Tuning switches of a context (tests and experiments; the defaults are the fastest
 * measured forms).  Unknown options or values return EDEN_ERR_INVALID_ARG.
 *   EDEN_OPT_PLAN_VARIANT  0 (default): no thread-block clusters; 1..3: an 8-block cluster
 *                          stage on the column pass, on the row pass, or on both, which
 *                          saves one sweep over HBM for 2^24..2^27 coordinates.
 *   EDEN_OPT_ROW_STAGING   1: the sender's last pass runs as a persistent kernel whose
 *                          tiles are staged in shared memory by bulk asynchronous copies.
 *   EDEN_OPT_SEL_ROUNDS    How the threshold of a b < 1 mask (the k-th smallest key) is found.
 *                          1 (default): in one pass over the keys, which keeps the keys inside
 *                          a band predicted from k/d as candidates; a job whose threshold
 *                          turns out to lie outside its band is redone by form 2 (the mask is
 *                          the same either way).  2: a histogram pass, then the candidate
 *                          pass.  3: three histogram rounds (the form vectors too long for
 *                          the candidate list use whatever this option says).
 *   EDEN_OPT_SEL_BAND      Half-width of form 1's band in tenths of a standard deviation of
 *                          the k-th smallest of d uniform keys, 0..120 (default 40).  0 leaves
 *                          the band empty, so every job is redone: for tests.
 *   EDEN_OPT_SLAB_MIB      0 (default): every pass of the transform is one launch over all
 *                          clients of a group; m > 0: vectors that take three sweeps run
 *                          their middle and last (receiver: first and middle) pass slab by
 *                          slab, m MiB of intermediate per slab, so that the second pass
 *                          of a slab may find the first one's output in the L2 cache. */
#define EDEN_OPT_PLAN_VARIANT 1
#define EDEN_OPT_ROW_STAGING  2
#define EDEN_OPT_SEL_ROUNDS   3
#define EDEN_OPT_SLAB_MIB     4
#define EDEN_OPT_SLAB_SIDES   6   /* 1: sender only, 2: receiver only, 3 (default): both */
#define EDEN_OPT_SEL_BAND     7
#define EDEN_OPT_SEL_AHEAD    8   /* 1 (default): in a call that mixes budgets below and above one bit, the masks of the
                                     b < 1 senders are selected on a side stream while the other senders' passes run on
                                     the context's stream, which waits for them where it needs them; 0: in line */
#define EDEN_OPT_SLAB_STREAMS 5   /* 1 (default)..4: slabs are dealt round-robin to this many streams, so that
                                     one slab's second pass can overlap the next slab's first */
int eden_set_option(eden_ctx* ctx, int option, int value);

/* Host only, no GPU: the band of 32-bit keys [*lo, *hi] in which form 1 of the mask
 * selection (EDEN_OPT_SEL_ROUNDS) expects the threshold of a mask that keeps k of d
 * coordinates (Section 4.1: a sample of exactly d*p coordinates; the keys that rank them
 * are uniform 32-bit words), `tenths` being EDEN_OPT_SEL_BAND's value.  *lo > *hi: no
 * prediction (the band would not fit the candidate list, or tenths = 0).  Returns
 * EDEN_ERR_INVALID_ARG for k = 0, k > d, tenths outside 0..120 or null pointers. */
int eden_mask_threshold_band(uint64_t d, uint64_t k, int tenths, uint32_t* lo, uint32_t* hi);

/* Optional per-kernel timing for benchmarks: while enabled, every kernel launch is
 * bracketed by CUDA events on the context's stream.  eden_profile_collect synchronises
 * and folds the records since eden_profile_enable(ctx, 1) into one entry per kernel
 * name; eden_profile_get returns entry i: launches, summed event time (ms) and summed
 * algorithmic bytes (what the step must read and write, not what it happened to move). */
int eden_profile_enable(eden_ctx* ctx, int on);
int eden_profile_collect(eden_ctx* ctx, uint32_t* n_kernels);
int eden_profile_get(eden_ctx* ctx, uint32_t i, const char** name, uint64_t* launches,
                     double* ms_total, double* bytes_total);
const char* eden_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* EDEN_H_ */
