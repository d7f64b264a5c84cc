/*
 * EDEN reference oracle (CPU, plain C, double precision).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct statement of
 * what the GPU library must compute.  It shares no code, table or constant generator
 * with the CUDA path and must never be linked into, imported by or called from it.
 * Only the test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it follows (arXiv 2108.08842, "EDEN"):
 *   - Section 2.2.1: sender = rotate, quantise eta_x * R(x) with a deterministic
 *     quantiser Q, eta_x = sqrt(d)/||x||_2.
 *   - Section 2.3:   scale S = ||x||^2 / <R(x), Q(eta_x R(x))>.
 *   - Section 2.2.2: receiver x_hat = S * R^-1(Q(...)); estimate = mean over senders.
 *   - Section 3:     Q's values are the Lloyd-Max centres of mass for N(0,1), 2^b levels.
 *   - Section 4.1:   b < 1: random sparsification mask of exact size d*p, factor 1/p,
 *                    applied before the rotation, then 1-bit EDEN.
 *   - Section 4.2:   lost rotated coordinates count as 0, multiply by 1/p,
 *                    p = received fraction (Lemma 4.3).
 *   - Section 5:     the rotation is the randomized Hadamard transform
 *                    R = (1/sqrt D) H_D Diag(s).
 *
 * Conventions the paper leaves open (all are readings chosen by this implementation; the ones marked
 * [unpinned] are pinned only by oracle == GPU):
 *   - H is the Sylvester matrix H[i][j] = (-1)^popcount(i & j); one transform.
 *   - d that is not a power of two is zero-padded to D = 2^ceil(log2 d'); all D
 *     rotated coordinates are coded; the estimate is truncated back.
 *   - Shared randomness is Philox4x32-10 (Salmon et al., SC'11), key = the 64-bit
 *     seed, counter = (call index lo, hi, stream id, 0).            [stream layout unpinned]
 *       stream 0, call t: 128 sign bits of rotated coordinates 128t..128t+127,
 *                         coordinate i -> word (i/32)%4, bit i%32, 1 means -1.
 *       stream 1, call t: the 32-bit mask keys of input coordinates 4t..4t+3.
 *   - Sub-bit mask: keep the k = floor(d*b + 0.5) (at least 1) coordinates with the
 *     smallest (key, index) pairs; p = k/d exactly.
 *   - An endpoint belongs to the interval nearer zero (Section 2.2.1, footnote);
 *     z = +-0 goes to the non-negative side.                         [tie at 0 unpinned]
 *   - Code of a coordinate = rank of its centroid in ascending order.
 *   - Wire layout: the codes form one little-endian bit stream of W-bit fields,
 *     coordinate i in stream bits [i*W, i*W + W) (bit b of the stream = bit b%32
 *     of 32-bit word b/32), low bit of the code first.                [layout unpinned]
 *   - A packet is 1024 consecutive rotated coordinates.
 *   - Non-integer budgets b > 1 (Section 4.1): coordinate i is coded with 2^(floor(b)+1)
 *     values if its coin is set, else with 2^floor(b).  Coins are Philox stream 2:
 *     call t yields sixteen 8-bit numbers (the bytes of word 0 from the low one up,
 *     then those of word 1, ...) for rotated coordinates 16t..16t+15; the coin is set
 *     iff the number is below round((b - floor(b)) * 256).            [stream layout unpinned]
 *     Wire layout for such b: groups of 32 coordinates, floor(b)+1 words each: first a
 *     bit stream of floor(b)-bit fields (the code of an unset coordinate, or the
 *     upper floor(b) bits of a set coordinate's code), then one word whose bit l is the
 *     lowest code bit of coordinate l of the group if its coin is set, else 0.
 *     Only floor(b)*32 + (number of coins) bits of a group carry information (both
 *     sides know the coins); the group keeps whole words so that packets keep
 *     their size.                                                      [layout unpinned]
 *   - Section 4.3's uniform-interval family I_Delta (functions *_uniform_* at the end):
 *     index n = round(z / Delta), an endpoint going to the interval nearer zero like
 *     everywhere else; indices are clamped to +-127, i.e. the family is made finite by
 *     letting the two outermost intervals run to infinity; the message is one signed
 *     byte per rotated coordinate (what an entropy coder would consume; the coder itself
 *     is not implemented here) plus S.  Boundary k is fl32(fl32(Delta) * (k - 1/2)).
 *                                                       [clamp, byte layout unpinned]
 *   - The interval decision is taken after rounding z and the boundary to fp32,
 *     the precision the GPU kernels decide in; everything else is double.
 *   - ||x|| = 0: scale 0, all codes 0.  A client with no received packet
 *     contributes nothing; the mean still divides by n.
 *
 * Parity unpinned (by the paper): the wire layout, the Philox stream layout and the
 * tie-breaks above.  Everything else is pinned by tests/test_oracle_*.py.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define EDEN_ORACLE_PACKET 1024u

/* ------------------------------------------------------------------------- */
/* Philox4x32-10, as published (Salmon, Moraes, Dror, Shaw; SC'11).           */
/* ------------------------------------------------------------------------- */
void eden_oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2], uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { /* Weyl key schedule between rounds */
            k0 += 0x9E3779B9u;
            k1 += 0xBB67AE85u;
        }
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static void philox_stream(uint64_t seed, uint32_t stream, uint64_t call, uint32_t out[4])
{
    uint32_t ctr[4] = { (uint32_t)call, (uint32_t)(call >> 32), stream, 0u };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    eden_oracle_philox4x32_10(ctr, key, out);
}

/* sign of rotated coordinate i: +1 or -1 (stream 0) */
double eden_oracle_sign(uint64_t seed, uint64_t i)
{
    uint32_t w[4];
    philox_stream(seed, 0u, i / 128u, w);
    uint32_t bit = (w[(i / 32u) % 4u] >> (i % 32u)) & 1u;
    return bit ? -1.0 : 1.0;
}

/* mask key of input coordinate i (stream 1) */
uint32_t eden_oracle_mask_key(uint64_t seed, uint64_t i)
{
    uint32_t w[4];
    philox_stream(seed, 1u, i / 4u, w);
    return w[i % 4u];
}

/* ------------------------------------------------------------------------- */
/* Size rules                                                                 */
/* ------------------------------------------------------------------------- */
uint64_t eden_oracle_kept_count(uint64_t d, double bits)
{
    if (bits >= 1.0) return d;
    uint64_t k = (uint64_t)floor((double)d * bits + 0.5);
    if (k < 1) k = 1;
    if (k > d) k = d;
    return k;
}

uint64_t eden_oracle_rot_dim(uint64_t d, double bits)
{
    uint64_t dp = eden_oracle_kept_count(d, bits);
    uint64_t D = 1;
    while (D < dp) D <<= 1;
    return D;
}

/* widest code of a client: 1 for b <= 1, b for integer b, floor(b)+1 otherwise */
uint32_t eden_oracle_code_width(double bits)
{
    if (bits <= 1.0) return 1u;
    if (bits == floor(bits)) return (uint32_t)bits;
    return (uint32_t)floor(bits) + 1u;
}

/* 0 for an integer (or sub-bit) budget, else the coin threshold round(frac * 256) in 1..255 */
uint32_t eden_oracle_coin_threshold(double bits)
{
    if (bits <= 1.0 || bits == floor(bits)) return 0u;
    uint32_t t = (uint32_t)floor((bits - floor(bits)) * 256.0 + 0.5);
    if (t < 1u) t = 1u;
    if (t > 255u) t = 255u;
    return t;
}

/* coin of rotated coordinate i for a non-integer budget (Philox stream 2) */
int eden_oracle_coin(uint64_t seed, uint64_t i, uint32_t threshold)
{
    uint32_t w[4];
    philox_stream(seed, 2u, i / 16u, w);
    uint32_t word = w[(i % 16u) / 4u];
    uint32_t byte = (word >> (8u * (uint32_t)(i % 4u))) & 0xFFu;
    return byte < threshold;
}

/* words of one client's message */
uint64_t eden_oracle_code_words(uint64_t D, double bits)
{
    uint32_t W = eden_oracle_code_width(bits);
    if (eden_oracle_coin_threshold(bits)) return ((D + 31u) / 32u) * W;   /* padded groups */
    return (D * W + 31u) / 32u;
}

/* ------------------------------------------------------------------------- */
/* Lloyd-Max quantiser for N(0,1) with n_levels values (Section 3).            */
/* Fixed point of:  boundary = midpoint of neighbouring values (nearest-value  */
/* rule, Section 3) and value = centre of mass of its interval (Section 2.2.1) */
/*   q_I = (phi(a) - phi(a')) / (Phi(a') - Phi(a))  for I = [a, a'].           */
/* centroids[n_levels] ascending; boundaries[n_levels-1] ascending.            */
/* Returns the number of iterations used.                                      */
/* ------------------------------------------------------------------------- */
static double std_normal_pdf(double t)
{
    if (isinf(t)) return 0.0;
    return exp(-0.5 * t * t) / sqrt(2.0 * M_PI);
}

/* P[a <= z <= a'] without cancellation in the tails */
static double std_normal_mass(double a, double b)
{
    if (a >= 0.0) return 0.5 * (erfc(a / M_SQRT2) - erfc(b / M_SQRT2));
    if (b <= 0.0) return 0.5 * (erfc(-b / M_SQRT2) - erfc(-a / M_SQRT2));
    return 0.5 * (erf(b / M_SQRT2) - erf(a / M_SQRT2));
}

double eden_oracle_interval_mass(double a, double b) { return std_normal_mass(a, b); }

double eden_oracle_centre_of_mass(double a, double b)
{
    return (std_normal_pdf(a) - std_normal_pdf(b)) / std_normal_mass(a, b);
}

int eden_oracle_lloyd_max(uint32_t n_levels, double *centroids, double *boundaries)
{
    /* the change per sweep stalls near 3e-14 (rounding of erfc/exp at 256 levels), so
       stop at 1e-13; the fixed-point residual is what the tests pin */
    const int max_iter = 1000000;
    uint32_t n = n_levels;
    if (n == 1) { centroids[0] = 0.0; return 0; }
    /* start from equal-probability-ish spread, symmetric */
    for (uint32_t j = 0; j < n; ++j)
        centroids[j] = -3.0 + 6.0 * ((double)j + 0.5) / (double)n;
    int it = 0;
    for (; it < max_iter; ++it) {
        for (uint32_t j = 0; j + 1 < n; ++j)
            boundaries[j] = 0.5 * (centroids[j] + centroids[j + 1]);
        double change = 0.0;
        for (uint32_t j = 0; j < n; ++j) {
            double a = (j == 0) ? -INFINITY : boundaries[j - 1];
            double b = (j + 1 == n) ? INFINITY : boundaries[j];
            double c = eden_oracle_centre_of_mass(a, b);
            double delta = fabs(c - centroids[j]);
            if (delta > change) change = delta;
            centroids[j] = c;
        }
        /* the density is even, so the unique fixed point is symmetric: enforce it */
        for (uint32_t j = 0; j < n / 2; ++j) {
            double m = 0.5 * (centroids[n - 1 - j] - centroids[j]);
            centroids[j] = -m;
            centroids[n - 1 - j] = m;
        }
        if (n % 2 == 1) centroids[n / 2] = 0.0;
        if (change < 1e-13) { ++it; break; }
    }
    for (uint32_t j = 0; j + 1 < n; ++j)
        boundaries[j] = 0.5 * (centroids[j] + centroids[j + 1]);
    if (n % 2 == 0) boundaries[n / 2 - 1] = 0.0;
    return it;
}

/* cache of the 2^W tables, W = 1..8 */
static double g_cent[9][256];
static double g_bound[9][255];
static int g_have[9];

static void table_for_width(uint32_t W, const double **cent, const double **bound)
{
    if (!g_have[W]) {
        /* solve into locals and publish afterwards: two threads that both find the cache
           empty then store identical tables instead of one reading a half-built one */
        double c[256], b[255];
        eden_oracle_lloyd_max(1u << W, c, b);
        memcpy(g_cent[W], c, sizeof(double) * (1u << W));
        memcpy(g_bound[W], b, sizeof(double) * ((1u << W) - 1u));
        g_have[W] = 1;
    }
    *cent = g_cent[W];
    *bound = g_bound[W];
}

void eden_oracle_table(uint32_t W, double *centroids, double *boundaries)
{
    const double *c, *b;
    table_for_width(W, &c, &b);
    memcpy(centroids, c, sizeof(double) * (1u << W));
    memcpy(boundaries, b, sizeof(double) * ((1u << W) - 1u));
}

/* ------------------------------------------------------------------------- */
/* Interval rule of Section 2.2.1 for one normalised coordinate z.            */
/* Magnitude index m = number of positive boundaries strictly below |z|       */
/* (an endpoint goes to the interval nearer zero); z >= 0 (including -0.0)    */
/* takes the upper half.  code = rank of the value in ascending order.        */
/* The comparison is done on fp32-rounded operands (see header).              */
/* ------------------------------------------------------------------------- */
uint32_t eden_oracle_quantise(double z, uint32_t W)
{
    const double *cent, *bound;
    table_for_width(W, &cent, &bound);
    uint32_t half = 1u << (W - 1);
    float az = (float)fabs(z);
    uint32_t m = 0;
    for (uint32_t j = 0; j + 1 < half; ++j) {
        float t = (float)bound[half + j]; /* positive boundaries, ascending */
        if (az > t) ++m;
    }
    int neg = (z < 0.0);
    return neg ? (half - 1u - m) : (half + m);
}

double eden_oracle_value(uint32_t code, uint32_t W)
{
    const double *cent, *bound;
    table_for_width(W, &cent, &bound);
    return cent[code];
}

/* ------------------------------------------------------------------------- */
/* Walsh-Hadamard transform, unnormalised, Sylvester order, in place.         */
/* Stages with strides 1, 2, 4, ..., D/2; pair (a, b) -> (a + b, a - b).      */
/* ------------------------------------------------------------------------- */
void eden_oracle_fwht(double *v, uint64_t D)
{
    for (uint64_t h = 1; h < D; h <<= 1)
        for (uint64_t base = 0; base < D; base += 2 * h)
            for (uint64_t j = base; j < base + h; ++j) {
                double a = v[j], b = v[j + h];
                v[j] = a + b;
                v[j + h] = a - b;
            }
}

/* One entry of H_D v straight from the definition H[i][j] = (-1)^popcount(i&j). */
double eden_oracle_hadamard_row_dot(const double *v, uint64_t D, uint64_t i)
{
    double acc = 0.0;
    for (uint64_t j = 0; j < D; ++j)
        acc += (__builtin_popcountll(i & j) & 1) ? -v[j] : v[j];
    return acc;
}

/* ------------------------------------------------------------------------- */
/* Sub-bit mask (Section 4.1): exactly k ones, uniformly random through the   */
/* shared seed: the k smallest (key, index) pairs.  mask[d] bytes of 0/1.     */
/* ------------------------------------------------------------------------- */
typedef struct { uint32_t key; uint64_t idx; } key_idx;

static int cmp_key_idx(const void *pa, const void *pb)
{
    const key_idx *a = (const key_idx *)pa, *b = (const key_idx *)pb;
    if (a->key != b->key) return a->key < b->key ? -1 : 1;
    if (a->idx != b->idx) return a->idx < b->idx ? -1 : 1;
    return 0;
}

int eden_oracle_mask(uint64_t seed, uint64_t d, uint64_t k, uint8_t *mask)
{
    key_idx *p = (key_idx *)malloc(sizeof(key_idx) * d);
    if (!p) return -1;
    for (uint64_t i = 0; i < d; ++i) { p[i].key = eden_oracle_mask_key(seed, i); p[i].idx = i; }
    qsort(p, d, sizeof(key_idx), cmp_key_idx);
    memset(mask, 0, d);
    for (uint64_t j = 0; j < k; ++j) mask[p[j].idx] = 1;
    free(p);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Sender (Sections 2.2.1, 2.3, 4.1).                                         */
/*   x[d] fp32 input, bits = budget b, seed = shared seed.                    */
/*   codes: D*W/32 words (layout in the header).  scale_out: S (double).      */
/*   z_out (optional, D doubles): the normalised rotated coordinates, so a    */
/*   caller can tell which coordinates sit next to an interval boundary.      */
/*   mask_out (optional, d bytes): the sparsification mask used (all 1 if     */
/*   b >= 1).  Returns 0, or -1 on allocation failure.                        */
/* ------------------------------------------------------------------------- */
int eden_oracle_encode(const float *x, uint64_t d, double bits, uint64_t seed,
                       uint32_t *codes, double *scale_out, double *z_out, uint8_t *mask_out)
{
    uint64_t k = eden_oracle_kept_count(d, bits);
    uint64_t D = eden_oracle_rot_dim(d, bits);
    uint32_t W = eden_oracle_code_width(bits);
    uint64_t n_words = eden_oracle_code_words(D, bits);
    uint32_t coin_thr = eden_oracle_coin_threshold(bits);
    uint32_t W0 = coin_thr ? W - 1u : W;       /* width of the fixed fields */

    double *y = (double *)calloc(D, sizeof(double));
    if (!y) return -1;

    /* step 1: y = sparsified, rescaled, compacted input, zero-padded to D */
    if (bits < 1.0) {
        uint8_t *mask = (uint8_t *)malloc(d);
        if (!mask) { free(y); return -1; }
        if (eden_oracle_mask(seed, d, k, mask)) { free(mask); free(y); return -1; }
        double inv_p = (double)d / (double)k;
        uint64_t j = 0;
        for (uint64_t i = 0; i < d; ++i)
            if (mask[i]) y[j++] = (double)x[i] * inv_p;
        if (mask_out) memcpy(mask_out, mask, d);
        free(mask);
    } else {
        for (uint64_t i = 0; i < d; ++i) y[i] = (double)x[i];
        if (mask_out) memset(mask_out, 1, d);
    }

    /* step 2: ||y||^2 */
    double N2 = 0.0;
    for (uint64_t i = 0; i < D; ++i) N2 += y[i] * y[i];

    memset(codes, 0, sizeof(uint32_t) * n_words);
    if (N2 == 0.0) {
        *scale_out = 0.0;
        if (z_out) memset(z_out, 0, sizeof(double) * D);
        free(y);
        return 0;
    }

    /* step 3: r = R(y) = (1/sqrt D) H Diag(s) y */
    for (uint64_t i = 0; i < D; ++i) y[i] *= eden_oracle_sign(seed, i);
    eden_oracle_fwht(y, D);
    double inv_sqrt_D = 1.0 / sqrt((double)D);
    for (uint64_t i = 0; i < D; ++i) y[i] *= inv_sqrt_D; /* y now holds r */

    /* steps 4-6: z = eta r with eta = sqrt(D)/||y||, code, dot <r, Q(z)> */
    double eta = sqrt((double)D) / sqrt(N2);
    double dot = 0.0;
    for (uint64_t i = 0; i < D; ++i) {
        double z = eta * y[i];
        if (!coin_thr) {
            uint32_t code = eden_oracle_quantise(z, W);
            dot += y[i] * eden_oracle_value(code, W);
            for (uint32_t j = 0; j < W; ++j) {           /* field i of the bit stream */
                uint64_t b = i * W + j;
                codes[b / 32u] |= ((code >> j) & 1u) << (b % 32u);
            }
        } else {
            /* non-integer budget: 2^(W0+1) values if the coin is set, else 2^W0 */
            uint64_t g = i / 32u, l = i % 32u;
            uint32_t *grp = codes + g * W;
            int coin = eden_oracle_coin(seed, i, coin_thr);
            uint32_t Wi = coin ? W0 + 1u : W0;
            uint32_t code = eden_oracle_quantise(z, Wi);
            dot += y[i] * eden_oracle_value(code, Wi);
            uint32_t field = coin ? code >> 1 : code;
            for (uint32_t j = 0; j < W0; ++j) {
                uint64_t b = l * W0 + j;
                grp[b / 32u] |= ((field >> j) & 1u) << (b % 32u);
            }
            if (coin) grp[W0] |= (code & 1u) << l;
        }
        if (z_out) z_out[i] = z;
    }
    *scale_out = N2 / dot;
    free(y);
    return 0;
}

/* number of 1024-coordinate packets of a D-vector */
uint64_t eden_oracle_num_packets(uint64_t D)
{
    return (D + EDEN_ORACLE_PACKET - 1u) / EDEN_ORACLE_PACKET;
}

/* ------------------------------------------------------------------------- */
/* Receiver, one sender (Sections 2.2.2, 4.1, 4.2).                           */
/*   recv_mask: bit i of word i/32 = packet i arrived; NULL = nothing lost.   */
/*   xhat[d] is overwritten with the estimate of this sender's vector.        */
/*   Returns 0; 1 if no packet arrived (xhat = 0); -1 on allocation failure.  */
/* ------------------------------------------------------------------------- */
int eden_oracle_decode(const uint32_t *codes, double S, double bits, uint64_t seed,
                       const uint32_t *recv_mask, uint64_t d, double *xhat)
{
    uint64_t k = eden_oracle_kept_count(d, bits);
    uint64_t D = eden_oracle_rot_dim(d, bits);
    uint32_t W = eden_oracle_code_width(bits);
    uint32_t coin_thr = eden_oracle_coin_threshold(bits);
    uint32_t W0 = coin_thr ? W - 1u : W;

    memset(xhat, 0, sizeof(double) * d);
    double *q = (double *)calloc(D, sizeof(double));
    if (!q) return -1;

    uint64_t received = 0;
    for (uint64_t i = 0; i < D; ++i) {
        uint64_t pkt = i / EDEN_ORACLE_PACKET;
        int arrived = recv_mask ? (int)((recv_mask[pkt / 32u] >> (pkt % 32u)) & 1u) : 1;
        if (coin_thr) {
            uint64_t g = i / 32u, l = i % 32u;
            const uint32_t *grp = codes + g * W;
            int coin = eden_oracle_coin(seed, i, coin_thr);
            if (!arrived) continue;
            ++received;
            uint32_t field = 0;
            for (uint32_t j = 0; j < W0; ++j) {
                uint64_t b = l * W0 + j;
                field |= ((grp[b / 32u] >> (b % 32u)) & 1u) << j;
            }
            if (coin) q[i] = eden_oracle_value((field << 1) | ((grp[W0] >> l) & 1u), W0 + 1u);
            else q[i] = eden_oracle_value(field, W0);
            continue;
        }
        if (!arrived) continue; /* lost coordinate counts as 0 */
        ++received;
        uint32_t code = 0;
        for (uint32_t j = 0; j < W; ++j) {
            uint64_t b = i * W + j;
            code |= ((codes[b / 32u] >> (b % 32u)) & 1u) << j;
        }
        q[i] = eden_oracle_value(code, W);
    }
    if (received == 0) { free(q); return 1; }
    double p = (double)received / (double)D;

    /* R^-1(q) = Diag(s) (1/sqrt D) H q, then the scale S and the loss factor 1/p */
    eden_oracle_fwht(q, D);
    double f = S / (p * sqrt((double)D));
    for (uint64_t i = 0; i < D; ++i) q[i] *= f * eden_oracle_sign(seed, i);

    if (bits < 1.0) {
        uint8_t *mask = (uint8_t *)malloc(d);
        if (!mask) { free(q); return -1; }
        if (eden_oracle_mask(seed, d, k, mask)) { free(mask); free(q); return -1; }
        uint64_t j = 0;
        for (uint64_t i = 0; i < d; ++i)
            if (mask[i]) xhat[i] = q[j++];
        free(mask);
    } else {
        for (uint64_t i = 0; i < d; ++i) xhat[i] = q[i];
    }
    free(q);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Section 4.1, the other order: sparsify AFTER the rotation.                  */
/* The sender rotates and codes the whole vector with one bit per coordinate   */
/* exactly as for b = 1 (same S), then sends only the coordinates of a random  */
/* mask over the D ROTATED coordinates: exactly k' = floor(D b + 1/2) ones,    */
/* the k' smallest (key, index) pairs of the shared seed's mask keys, now      */
/* indexed by the rotated coordinate.  The message is the sign bits of the     */
/* kept coordinates in increasing index order (k' bits).  The receiver puts 0  */
/* for the others and multiplies by 1/p, p = k'/D, which is Lemma 4.3 with     */
/* this mask as the deterministic one.           [mask rule and layout unpinned] */
/* ------------------------------------------------------------------------- */
uint64_t eden_oracle_after_kept_count(uint64_t d, double bits)
{
    uint64_t D = eden_oracle_rot_dim(d, 1.0);
    return eden_oracle_kept_count(D, bits);
}

int eden_oracle_encode_after(const float *x, uint64_t d, double bits, uint64_t seed,
                             uint32_t *codes, double *scale_out, double *z_out, uint8_t *mask_out)
{
    uint64_t D = eden_oracle_rot_dim(d, 1.0);
    uint64_t k = eden_oracle_after_kept_count(d, bits);
    double *y = (double *)calloc(D, sizeof(double));
    uint8_t *mask = (uint8_t *)malloc(D);
    if (!y || !mask) { free(y); free(mask); return -1; }
    if (eden_oracle_mask(seed, D, k, mask)) { free(y); free(mask); return -1; }
    if (mask_out) memcpy(mask_out, mask, D);
    for (uint64_t i = 0; i < d; ++i) y[i] = (double)x[i];
    double N2 = 0.0;
    for (uint64_t i = 0; i < D; ++i) N2 += y[i] * y[i];
    memset(codes, 0, sizeof(uint32_t) * ((k + 31u) / 32u));
    if (N2 == 0.0) {
        *scale_out = 0.0;
        if (z_out) memset(z_out, 0, sizeof(double) * D);
        free(y); free(mask);
        return 0;
    }
    for (uint64_t i = 0; i < D; ++i) y[i] *= eden_oracle_sign(seed, i);
    eden_oracle_fwht(y, D);
    double inv_sqrt_D = 1.0 / sqrt((double)D);
    for (uint64_t i = 0; i < D; ++i) y[i] *= inv_sqrt_D;          /* r = R(x) */
    double eta = sqrt((double)D) / sqrt(N2);
    double dot = 0.0;
    uint64_t j = 0;                                               /* next bit of the message */
    for (uint64_t i = 0; i < D; ++i) {
        double z = eta * y[i];
        uint32_t code = eden_oracle_quantise(z, 1);
        dot += y[i] * eden_oracle_value(code, 1);                 /* over ALL coordinates: S as for b = 1 */
        if (mask[i]) {
            codes[j / 32u] |= code << (j % 32u);
            ++j;
        }
        if (z_out) z_out[i] = z;
    }
    *scale_out = N2 / dot;
    free(y); free(mask);
    return 0;
}

int eden_oracle_decode_after(const uint32_t *codes, double S, double bits, uint64_t seed,
                             uint64_t d, double *xhat)
{
    uint64_t D = eden_oracle_rot_dim(d, 1.0);
    uint64_t k = eden_oracle_after_kept_count(d, bits);
    double *q = (double *)calloc(D, sizeof(double));
    uint8_t *mask = (uint8_t *)malloc(D);
    if (!q || !mask) { free(q); free(mask); return -1; }
    if (eden_oracle_mask(seed, D, k, mask)) { free(q); free(mask); return -1; }
    uint64_t j = 0;
    for (uint64_t i = 0; i < D; ++i)
        if (mask[i]) {
            q[i] = eden_oracle_value((codes[j / 32u] >> (j % 32u)) & 1u, 1);
            ++j;
        }
    double p = (double)k / (double)D;
    eden_oracle_fwht(q, D);
    double f = S / (p * sqrt((double)D));
    for (uint64_t i = 0; i < d; ++i) xhat[i] = q[i] * f * eden_oracle_sign(seed, i);
    free(q); free(mask);
    return 0;
}

/* ------------------------------------------------------------------------- */
/* Section 4.3: the uniform-interval family                                    */
/*   I_Delta = { [Delta (n - 1/2), Delta (n + 1/2)] : n integer },             */
/* its entropy H = -sum_n p_n log2 p_n under N(0,1), Delta_b = the smallest    */
/* Delta with H <= b, and EDEN with Q = centre of mass of the interval.        */
/* ------------------------------------------------------------------------- */
#define EDEN_ORACLE_UNIFORM_MAX_INDEX 127

double eden_oracle_uniform_entropy(double delta)
{
    double p0 = std_normal_mass(-0.5 * delta, 0.5 * delta);
    double h = p0 > 0.0 ? -p0 * log2(p0) : 0.0;
    for (uint64_t n = 1;; ++n) {
        double a = delta * ((double)n - 0.5);
        double p = std_normal_mass(a, a + delta);
        if (!(p > 0.0)) break;                 /* the tail mass has underflowed */
        h -= 2.0 * p * log2(p);                /* intervals n and -n */
    }
    return h;
}

/* H falls as Delta grows, so "the smallest Delta with H <= b" is the root of H = b. */
double eden_oracle_uniform_delta(double bits)
{
    double lo = 1e-4, hi = 64.0;               /* H(lo) ~ 15.3 bits, H(hi) ~ 0 */
    if (!(bits > eden_oracle_uniform_entropy(hi)) || !(bits < eden_oracle_uniform_entropy(lo))) return 0.0;
    for (int it = 0; it < 200; ++it) {
        double mid = 0.5 * (lo + hi);
        if (eden_oracle_uniform_entropy(mid) <= bits) hi = mid; else lo = mid;
    }
    return hi;
}

/* centre of mass of the interval of magnitude index m (0 <= m <= 127); the index's sign
   is the value's sign                                     [underflow rule unpinned] */
double eden_oracle_uniform_value(double delta, uint32_t m)
{
    if (m == 0) return 0.0;
    double a = delta * ((double)m - 0.5);
    double b = m == EDEN_ORACLE_UNIFORM_MAX_INDEX ? INFINITY : a + delta;
    /* beyond ~38 standard deviations the mass underflows in double precision; such an
       interval (never reached by data) takes its inner endpoint as its value */
    if (!(std_normal_mass(a, b) > 0.0)) return a;
    return eden_oracle_centre_of_mass(a, b);
}

/* E[Q(z)^2] of the clamped family; vNMSE = 1/E[Q^2] - 1 (Corollary 2.4) */
double eden_oracle_uniform_second_moment(double delta)
{
    double acc = 0.0;
    for (uint32_t m = 1; m <= EDEN_ORACLE_UNIFORM_MAX_INDEX; ++m) {
        double a = delta * ((double)m - 0.5);
        double b = m == EDEN_ORACLE_UNIFORM_MAX_INDEX ? INFINITY : a + delta;
        double q = eden_oracle_uniform_value(delta, m);
        acc += 2.0 * std_normal_mass(a, b) * q * q;
    }
    return acc;
}

/* index of z: the number of positive boundaries Delta (k - 1/2), k = 1..127, strictly
   below |z|, with z's sign; compared in fp32 like eden_oracle_quantise */
int32_t eden_oracle_uniform_index(double z, double delta)
{
    float az = (float)fabs(z);
    float df = (float)delta;
    int32_t m = 0;
    for (int32_t k = 1; k <= EDEN_ORACLE_UNIFORM_MAX_INDEX; ++k) {
        float t = df * ((float)k - 0.5f);
        if (az > t) m = k; else break;
    }
    return z < 0.0 ? -m : m;
}

/* Sender with Q over I_Delta (b >= 1 shape: no sparsification).  index[D] signed bytes. */
int eden_oracle_encode_uniform(const float *x, uint64_t d, double delta, uint64_t seed,
                               int8_t *index, double *scale_out, double *z_out)
{
    uint64_t D = eden_oracle_rot_dim(d, 1.0);
    double *y = (double *)calloc(D, sizeof(double));
    if (!y) return -1;
    for (uint64_t i = 0; i < d; ++i) y[i] = (double)x[i];
    double N2 = 0.0;
    for (uint64_t i = 0; i < D; ++i) N2 += y[i] * y[i];
    memset(index, 0, D);
    if (N2 == 0.0) {
        *scale_out = 0.0;
        if (z_out) memset(z_out, 0, sizeof(double) * D);
        free(y);
        return 0;
    }
    for (uint64_t i = 0; i < D; ++i) y[i] *= eden_oracle_sign(seed, i);
    eden_oracle_fwht(y, D);
    double inv_sqrt_D = 1.0 / sqrt((double)D);
    for (uint64_t i = 0; i < D; ++i) y[i] *= inv_sqrt_D;             /* r = R(y) */
    double eta = sqrt((double)D) / sqrt(N2);
    double dot = 0.0;
    for (uint64_t i = 0; i < D; ++i) {
        double z = eta * y[i];
        int32_t n = eden_oracle_uniform_index(z, delta);
        double q = eden_oracle_uniform_value(delta, (uint32_t)(n < 0 ? -n : n));
        dot += y[i] * (n < 0 ? -q : q);
        index[i] = (int8_t)n;
        if (z_out) z_out[i] = z;
    }
    *scale_out = N2 / dot;
    free(y);
    return 0;
}

/* Receiver for one sender of the uniform family; same contract as eden_oracle_decode.
   An index byte of -128 never occurs in a message; it is read as -127. */
int eden_oracle_decode_uniform(const int8_t *index, double S, double delta, uint64_t seed,
                               const uint32_t *recv_mask, uint64_t d, double *xhat)
{
    uint64_t D = eden_oracle_rot_dim(d, 1.0);
    memset(xhat, 0, sizeof(double) * d);
    double *q = (double *)calloc(D, sizeof(double));
    if (!q) return -1;
    uint64_t received = 0;
    for (uint64_t i = 0; i < D; ++i) {
        uint64_t pkt = i / EDEN_ORACLE_PACKET;
        int arrived = recv_mask ? (int)((recv_mask[pkt / 32u] >> (pkt % 32u)) & 1u) : 1;
        if (!arrived) continue;
        ++received;
        int32_t n = index[i];
        uint32_t m = (uint32_t)(n < 0 ? -n : n);
        if (m > EDEN_ORACLE_UNIFORM_MAX_INDEX) m = EDEN_ORACLE_UNIFORM_MAX_INDEX;
        double v = eden_oracle_uniform_value(delta, m);
        q[i] = n < 0 ? -v : v;
    }
    if (received == 0) { free(q); return 1; }
    double p = (double)received / (double)D;
    eden_oracle_fwht(q, D);
    double f = S / (p * sqrt((double)D));
    for (uint64_t i = 0; i < d; ++i) xhat[i] = q[i] * f * eden_oracle_sign(seed, i);
    free(q);
    return 0;
}
