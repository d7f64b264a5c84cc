// C ABI of the EDEN hot path (declared in include/eden.h): argument checks, the pass
// plan, workspace carving and kernel launches.  All arithmetic runs in the kernels.
#include "../../include/eden.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "eden_device.cuh"
#include "kernels_generic.cuh"
#include "kernels_fast.cuh"
#include "kernels_select.cuh"
#include "lloyd_max.h"
#include "uniform_family.h"

static_assert(eden::kStatusTimeout == EDEN_STATUS_TIMEOUT, "status bit of the bounded waits");

using namespace eden;

// ------------------------------------------------------------------------------------
// size rules
// ------------------------------------------------------------------------------------
static int ceil_log2(uint64_t v)
{
    int l = 0;
    while ((1ull << l) < v) ++l;
    return l;
}

extern "C" uint64_t eden_kept_count(uint64_t d, double bits)
{
    if (bits >= 1.0) return d;
    uint64_t k = (uint64_t)std::floor((double)d * bits + 0.5);
    if (k < 1) k = 1;
    if (k > d) k = d;
    return k;
}

extern "C" uint64_t eden_rot_dim(uint64_t d, double bits)
{
    return 1ull << ceil_log2(eden_kept_count(d, bits));
}

extern "C" uint32_t eden_code_width(double bits)
{
    if (!(bits > 0.0)) return 0;
    if (bits <= 1.0) return 1;
    if (bits > 8.0) return 0;
    if (bits == std::floor(bits)) return (uint32_t)bits;
    return (uint32_t)std::floor(bits) + 1;     // non-integer: the wider of the two tables
}

// 0 for integer and sub-bit budgets, else round(frac(b) * 256) clamped to [1, 255]
static uint32_t coin_threshold(double bits)
{
    if (bits <= 1.0 || bits == std::floor(bits)) return 0;
    uint32_t t = (uint32_t)std::floor((bits - std::floor(bits)) * 256.0 + 0.5);
    return std::min(std::max(t, 1u), 255u);
}

extern "C" uint64_t eden_code_bytes(uint64_t d, double bits)
{
    const uint64_t D = eden_rot_dim(d, bits);
    const uint64_t W = eden_code_width(bits);
    // integer budgets: one bit stream; non-integer: groups of 32 coordinates padded to W words
    const uint64_t words = coin_threshold(bits) ? ((D + 31) / 32) * W : (D * W + 31) / 32;
    return (words * 4 + 15) / 16 * 16;
}

extern "C" uint64_t eden_num_packets(uint64_t d, double bits)
{
    return (eden_rot_dim(d, bits) + EDEN_PACKET_COORDS - 1) / EDEN_PACKET_COORDS;
}

extern "C" uint64_t eden_recv_mask_words(uint64_t d, double bits)
{
    return (eden_num_packets(d, bits) + 31) / 32;
}

// ------------------------------------------------------------------------------------
// quantiser tables (host copy, built once per process)
// ------------------------------------------------------------------------------------
namespace {

struct Tables {
    float pos_boundary[256];
    float pos_value[256];
    std::vector<float> centroids[9], boundaries[9];
    FmaTree tree[9];
    bool tree_exact;
    float2 cells[9 - kCellMinWidth][kCellMax];
    float cell_zmax[9];
    int cell_count[9];
};

// fma(a, b, c) rounded towards zero, for a in {0, 1} and operands whose exact sum fits a double
float fma_rz_host(float a, float b, float c)
{
    const double exact = (double)a * (double)b + (double)c;
    float f = (float)exact;
    if ((double)f != exact && std::fabs((double)f) > std::fabs(exact)) f = std::nextafterf(f, 0.f);
    return f;
}

// x and its two neighbours
void neighbours(double x, float out[3])
{
    const float f = (float)x;
    out[0] = std::nextafterf(f, -INFINITY);
    out[1] = f;
    out[2] = std::nextafterf(f, INFINITY);
}

// Constants of the multiply-add interval search (FmaTree) for W = 2..4 from the positive
// fp32 boundaries: every boundary the search forms must be bit-identical to -2^30 times the
// table's boundary, so each difference is picked among the rounded difference and its two
// neighbours, checked over all indicator combinations.  Returns false if no choice works.
bool build_fma_tree(int W, const float* pb, const float* pv, FmaTree& tr)
{
    std::memset(&tr, 0, sizeof(tr));
    const float big = 1073741824.f;                       // 2^30
    tr.big = big;
    float T[7];
    for (int j = 0; j + 1 < (1 << (W - 1)); ++j) T[j] = -big * pb[j];     // exact: a power of two
    if (W == 2) {
        tr.k_root = T[0];
        tr.v0 = pv[0];
        tr.dv = pv[1] - pv[0];
        return true;
    }
    if (W == 3) {
        tr.k_root = T[1];
        tr.b1 = T[0];
        float cand[3];
        neighbours((double)T[2] - (double)T[0], cand);
        for (float a : cand)
            if (fma_rz_host(1.f, a, T[0]) == T[2]) { tr.a1 = a; return true; }
        return false;
    }
    tr.k_root = T[3];
    tr.b1 = T[1];
    tr.b_lo = T[0];
    bool ok = false;
    float c1[3], cl[3], ch[3], cb[3];
    neighbours((double)T[5] - (double)T[1], c1);
    for (float a : c1)
        if (fma_rz_host(1.f, a, T[1]) == T[5]) { tr.a1 = a; ok = true; break; }
    if (!ok) return false;
    neighbours((double)T[2] - (double)T[0], cl);
    neighbours((double)T[6] - (double)T[4], ch);
    neighbours((double)T[4] - (double)T[0], cb);
    for (float a_lo : cl)
        for (float a_hi : ch)
            for (float db : cb) {
                float cd[3];
                neighbours((double)a_hi - (double)a_lo, cd);
                for (float da : cd) {
                    bool good = true;
                    for (int i2 = 0; i2 < 2 && good; ++i2)
                        for (int i1 = 0; i1 < 2 && good; ++i1) {
                            const float p = fma_rz_host((float)i2, da, a_lo), q = fma_rz_host((float)i2, db, T[0]);
                            good = fma_rz_host((float)i1, p, q) == T[4 * i2 + 2 * i1];
                        }
                    if (good) {
                        tr.a_lo = a_lo; tr.da = da; tr.db = db;
                        return true;
                    }
                }
            }
    return false;
}

// Cell table of the one-step interval search for code width W (see c_cells): false if a
// cell would hold two boundaries or the table does not fit.
bool build_cells(int W, const float* pb, float2* cells, float* zmax, int* count)
{
    const int n_bound = (1 << (W - 1)) - 1;
    const double K = (double)(1 << (W - 2));               // cells per unit
    const int n_cells = (int)std::floor((double)pb[n_bound - 1] * K) + 2;
    if (n_cells > kCellMax) return false;
    int j = 0;                                              // boundaries below the current cell
    for (int c = 0; c < n_cells; ++c) {
        const double lo = c / K, hi = (c + 1) / K;
        int inside = 0;
        float t_in = 0.f;
        while (j + inside < n_bound && (double)pb[j + inside] < hi) {
            if ((double)pb[j + inside] < lo) return false;  // not sorted
            t_in = pb[j + inside];
            ++inside;
        }
        if (inside > 1) return false;
        uint32_t bits = 4u * (uint32_t)j;
        float count_as_float;
        std::memcpy(&count_as_float, &bits, sizeof(float));
        cells[c].x = inside ? -1073741824.f * t_in : -3.0e38f;
        cells[c].y = count_as_float;
        j += inside;
    }
    if (j != n_bound) return false;
    *zmax = (float)((n_cells - 0.5) / K);                   // exact: a small multiple of a power of two
    *count = n_cells;
    return true;
}

const Tables& tables()
{
    static Tables t;
    static std::once_flag once;
    std::call_once(once, [] {
        std::memset(t.pos_boundary, 0, sizeof(t.pos_boundary));
        std::memset(t.pos_value, 0, sizeof(t.pos_value));
        for (int W = 1; W <= 8; ++W) {
            std::vector<double> c, b;
            lloyd_max_table(W, c, b);
            t.centroids[W].assign(c.begin(), c.end());
            t.boundaries[W].assign(b.begin(), b.end());
            const int half = 1 << (W - 1), off = half - 1;
            for (int j = 0; j < half; ++j) t.pos_value[off + j] = (float)c[half + j];
            for (int j = 0; j + 1 < half; ++j) t.pos_boundary[off + j] = (float)b[half + j];
        }
        t.tree_exact = true;
        std::memset(t.tree, 0, sizeof(t.tree));
        for (int W = 2; W <= 8; ++W) {
            const int off = (1 << (W - 1)) - 1;
            // the saturated multiply-adds need one unit in the last place of any boundary,
            // times 2^30, to be at least 1: no boundary below 2^-7
            t.tree_exact = t.tree_exact && t.pos_boundary[off] >= 0.0078125f;
            if (W <= 4) {
                t.tree_exact = build_fma_tree(W, t.pos_boundary + off, t.pos_value + off, t.tree[W]) && t.tree_exact;
            } else {
                // wider tables: the tree settles the top three bits of the index, i.e. it
                // searches the seven boundaries at the eighth points of the table
                float coarse[7];
                const int eighth = (1 << (W - 1)) / 8;
                for (int j = 0; j < 7; ++j) coarse[j] = t.pos_boundary[off + (j + 1) * eighth - 1];
                t.tree_exact = build_fma_tree(4, coarse, t.pos_value + off, t.tree[W]) && t.tree_exact;
            }
        }
        std::memset(t.cells, 0, sizeof(t.cells));
        std::memset(t.cell_zmax, 0, sizeof(t.cell_zmax));
        std::memset(t.cell_count, 0, sizeof(t.cell_count));
        for (int W = kCellMinWidth; W <= 8; ++W)
            t.tree_exact = build_cells(W, t.pos_boundary + (1 << (W - 1)) - 1, t.cells[W - kCellMinWidth],
                                       &t.cell_zmax[W], &t.cell_count[W]) && t.tree_exact;
    });
    return t;
}

uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

constexpr uint64_t kHistBytes = 2ull * 65536 * sizeof(uint32_t);

// fixed part of the workspace: status word, mask-selection scratch
struct FixedLayout {
    uint64_t status, sel, hist, chunks, end;
};

FixedLayout fixed_layout(uint64_t d_max)
{
    FixedLayout f;
    f.status = 0;
    f.sel = 256;
    f.hist = 512;
    f.chunks = f.hist + kHistBytes;
    const uint64_t n_chunks = (d_max + kSelChunk - 1) / kSelChunk;
    f.end = align_up(f.chunks + n_chunks * sizeof(unsigned long long), 256);
    return f;
}

uint64_t per_client_bytes() { return align_up(sizeof(ClientDesc), 16) + align_up(sizeof(ClientState), 16); }

}  // namespace

extern "C" uint64_t eden_workspace_bytes(uint64_t d_max, uint32_t n_batch)
{
    if (n_batch == 0) n_batch = 1;
    const uint64_t D = 1ull << ceil_log2(d_max ? d_max : 1);
    // per client: descriptors, one intermediate vector, and (b < 1) the mask-selection scratch
    const uint64_t n_chunks = (d_max + kSelChunk - 1) / kSelChunk;
    const uint64_t sel = 256 + kHistBytes + align_up(n_chunks * sizeof(unsigned long long), 256) + 256 +
                         align_up(n_chunks * (kSelChunk / 8), 256);   // the last term: mask bitmap
    // partial sums of the receiver's last pass when a round has too few tiles to fill the
    // GPU (sized for 148 SMs; a split that does not fit is simply not used)
    const uint64_t tiles = std::max<uint64_t>(1, D >> 13);
    const uint64_t rows = std::min<uint64_t>(std::min<uint64_t>(n_batch, 16), (296 + tiles - 1) / tiles);
    const uint64_t partials = rows >= 2 ? rows * align_up(d_max, 64) * sizeof(float) : 0;
    return fixed_layout(d_max).end + align_up(per_client_bytes() * n_batch, 256) + 1024 + partials +
           (uint64_t)n_batch * (align_up(D * sizeof(float), 256) + sel + 512 /* uniform-family values */);
}

extern "C" int eden_table(uint32_t W, float* centroids, float* boundaries)
{
    if (W < 1 || W > 8 || !centroids || !boundaries) return EDEN_ERR_INVALID_ARG;
    const Tables& t = tables();
    std::copy(t.centroids[W].begin(), t.centroids[W].end(), centroids);
    std::copy(t.boundaries[W].begin(), t.boundaries[W].end(), boundaries);
    return EDEN_OK;
}

extern "C" int eden_self_check(void)
{
    return tables().tree_exact ? EDEN_OK : EDEN_ERR_INVALID_ARG;
}

extern "C" double eden_uniform_entropy(double delta)
{
    return delta > 0.0 ? uniform_entropy(delta) : 0.0;
}

extern "C" double eden_uniform_delta(double bits) { return uniform_delta(bits); }

extern "C" int eden_uniform_values(double delta, float* values)
{
    if (!values) return EDEN_ERR_INVALID_ARG;
    if (!(delta >= kUniformMinDelta) || !(delta < kUniformMaxDelta)) return EDEN_ERR_UNSUPPORTED_BITS;
    uniform_values(delta, values);
    return EDEN_OK;
}

extern "C" uint64_t eden_uniform_index_bytes(uint64_t d) { return (eden_rot_dim(d, 1.0) + 15) / 16 * 16; }

extern "C" const char* eden_strerror(int code)
{
    switch (code) {
        case EDEN_OK: return "ok";
        case EDEN_ERR_INVALID_ARG: return "invalid argument";
        case EDEN_ERR_UNSUPPORTED_BITS: return "unsupported bit budget (0 < b <= 8) or interval width (1/16 <= Delta < 2)";
        case EDEN_ERR_CUDA: return "CUDA error";
        case EDEN_ERR_WORKSPACE: return "workspace too small";
        case EDEN_ERR_TOO_LARGE: return "dimension too large";
        default: return "unknown error";
    }
}

// ------------------------------------------------------------------------------------
// context
// ------------------------------------------------------------------------------------
struct ProfileRecord {
    const char* name;
    double bytes;                    // algorithmic bytes of this launch
    cudaEvent_t start, stop;
};

struct ProfileSummary {
    const char* name;
    uint64_t launches;
    double ms, bytes;
};

struct eden_ctx {
    int device;
    cudaStream_t stream;
    char* ws;
    uint64_t ws_bytes;
    uint64_t launches;
    std::vector<uint32_t> order;     // processing order of the last call: order[j] = client
    uint64_t states_off;             // where the last call put its ClientState array
    bool profiling;
    bool profile_open;               // profile_begin recorded a start event that profile_end must close
    bool force_generic;
    int plan_variant;
    int row_staging;                 // 1: the sender's row pass runs in its persistent, bulk-copy-staged form
    int sel_rounds;                  // 3: the b < 1 mask threshold is found in three histogram rounds at every size
    int sel_band;                    // half-width of the predicted band of the one-pass selection, tenths of a standard deviation
    int sel_ahead;                   // 1: the masks of a call's b < 1 clients are selected on a side stream while the b >= 1 groups run
    cudaStream_t sel_stream;         // that side stream (created on first use)
    std::vector<cudaEvent_t> sel_events;   // fork (0), join (1) and one per b < 1 group (2 + ...)
    int slab_mib;                    // > 0: middle and row pass are launched slab by slab (MiB of intermediate per slab)
    int slab_streams;                // slabs are dealt round-robin to this many streams (1 = the context's own)
    int slab_sides;                  // bit 0: the sender uses the slab order, bit 1: the receiver
    std::vector<cudaStream_t> side;  // side streams of the slab order
    std::vector<cudaEvent_t> slab_events;   // fork (0) and join (1 + stream) events of the slab order
    int sm_count;
    std::vector<ProfileRecord> records;
    std::vector<std::pair<cudaEvent_t, cudaEvent_t>> event_pool;
    std::vector<ProfileSummary> summary;
    // host-buffer entry points: side streams and events for overlapping copies with kernels
    cudaStream_t copy_in, copy_out;
    std::vector<cudaEvent_t> sync_events;
};

static void profile_begin(eden_ctx* ctx, const char* name, double bytes)
{
    ctx->profile_open = false;
    if (!ctx->profiling) return;
    ProfileRecord r;
    r.name = name;
    r.bytes = bytes;
    if (ctx->records.size() < ctx->event_pool.size()) {
        r.start = ctx->event_pool[ctx->records.size()].first;
        r.stop = ctx->event_pool[ctx->records.size()].second;
    } else {
        if (cudaEventCreate(&r.start) != cudaSuccess) return;
        if (cudaEventCreate(&r.stop) != cudaSuccess) {
            cudaEventDestroy(r.start);
            return;
        }
        ctx->event_pool.push_back({r.start, r.stop});
    }
    cudaEventRecord(r.start, ctx->stream);
    ctx->records.push_back(r);
    ctx->profile_open = true;
}

static void profile_end(eden_ctx* ctx)
{
    if (!ctx->profile_open) return;
    cudaEventRecord(ctx->records.back().stop, ctx->stream);
    ctx->profile_open = false;
}

#define CUDA_OK(expr)                                 \
    do {                                              \
        if ((expr) != cudaSuccess) return EDEN_ERR_CUDA; \
    } while (0)

// name and algorithmic bytes feed the optional per-kernel event timing (eden_profile_*)
#define LAUNCH(ctx, name, bytes, kernel, grid, block, smem, ...)             \
    do {                                                                     \
        profile_begin(ctx, name, (double)(bytes));                           \
        kernel<<<grid, block, smem, (ctx)->stream>>>(__VA_ARGS__);           \
        profile_end(ctx);                                                    \
        ++(ctx)->launches;                                                   \
        if (cudaGetLastError() != cudaSuccess) return EDEN_ERR_CUDA;         \
    } while (0)

extern "C" int eden_create(eden_ctx** out, int cuda_device, void* cuda_stream,
                           void* workspace_dev, uint64_t workspace_bytes)
{
    if (!out || !workspace_dev || ((uintptr_t)workspace_dev & 255u)) return EDEN_ERR_INVALID_ARG;
    if (workspace_bytes < fixed_layout(1).end) return EDEN_ERR_WORKSPACE;
    CUDA_OK(cudaSetDevice(cuda_device));
    eden_ctx* ctx = new (std::nothrow) eden_ctx();
    if (!ctx) return EDEN_ERR_INVALID_ARG;
    ctx->device = cuda_device;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->ws = (char*)workspace_dev;
    ctx->ws_bytes = workspace_bytes;
    ctx->launches = 0;
    ctx->states_off = 0;
    ctx->profiling = false;
    ctx->profile_open = false;
    ctx->copy_in = nullptr;
    ctx->copy_out = nullptr;
    ctx->force_generic = false;
    ctx->plan_variant = 0;
    ctx->row_staging = 0;
    ctx->sel_rounds = 1;
    ctx->sel_band = 40;
    ctx->sel_ahead = 1;
    ctx->sel_stream = nullptr;
    ctx->slab_mib = 0;
    ctx->slab_streams = 1;
    ctx->slab_sides = 3;
    ctx->sm_count = 0;
    if (cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, cuda_device) != cudaSuccess ||
        ctx->sm_count <= 0) {
        delete ctx;
        return EDEN_ERR_CUDA;
    }
    const Tables& t = tables();
    if (!t.tree_exact) {                      // cannot happen with the Lloyd-Max tables (eden_self_check)
        delete ctx;
        return EDEN_ERR_INVALID_ARG;
    }
    if (cudaMemcpyToSymbol(c_tree, t.tree, sizeof(t.tree)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_cells, t.cells, sizeof(t.cells)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_cell_zmax, t.cell_zmax, sizeof(t.cell_zmax)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_cell_count, t.cell_count, sizeof(t.cell_count)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_pos_boundary, t.pos_boundary, sizeof(t.pos_boundary)) != cudaSuccess ||
        cudaMemcpyToSymbol(c_pos_value, t.pos_value, sizeof(t.pos_value)) != cudaSuccess ||
        cudaMemsetAsync(ctx->ws, 0, 256, ctx->stream) != cudaSuccess ||
        cudaStreamSynchronize(ctx->stream) != cudaSuccess) {
        delete ctx;
        return EDEN_ERR_CUDA;
    }
    *out = ctx;
    return EDEN_OK;
}

extern "C" int eden_destroy(eden_ctx* ctx)
{
    if (!ctx) return EDEN_ERR_INVALID_ARG;
    for (auto& e : ctx->event_pool) {
        cudaEventDestroy(e.first);
        cudaEventDestroy(e.second);
    }
    for (cudaEvent_t e : ctx->sync_events) cudaEventDestroy(e);
    for (cudaStream_t st : ctx->side) cudaStreamDestroy(st);
    for (cudaEvent_t e : ctx->slab_events) cudaEventDestroy(e);
    for (cudaEvent_t e : ctx->sel_events) cudaEventDestroy(e);
    if (ctx->sel_stream) cudaStreamDestroy(ctx->sel_stream);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    delete ctx;
    return EDEN_OK;
}

extern "C" uint64_t eden_launch_count(const eden_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" int eden_force_generic_kernels(eden_ctx* ctx, int on)
{
    if (!ctx) return EDEN_ERR_INVALID_ARG;
    ctx->force_generic = on != 0;
    return EDEN_OK;
}

extern "C" int eden_set_option(eden_ctx* ctx, int option, int value)
{
    if (!ctx) return EDEN_ERR_INVALID_ARG;
    switch (option) {
        case EDEN_OPT_PLAN_VARIANT:
            if (value < 0 || value > 3) return EDEN_ERR_INVALID_ARG;
            ctx->plan_variant = value;
            return EDEN_OK;
        case EDEN_OPT_ROW_STAGING:
            if (value != 0 && value != 1) return EDEN_ERR_INVALID_ARG;
            ctx->row_staging = value;
            return EDEN_OK;
        case EDEN_OPT_SEL_ROUNDS:
            if (value < 1 || value > 3) return EDEN_ERR_INVALID_ARG;
            ctx->sel_rounds = value;
            return EDEN_OK;
        case EDEN_OPT_SEL_BAND:
            if (value < 0 || value > 120) return EDEN_ERR_INVALID_ARG;
            ctx->sel_band = value;
            return EDEN_OK;
        case EDEN_OPT_SEL_AHEAD:
            if (value != 0 && value != 1) return EDEN_ERR_INVALID_ARG;
            ctx->sel_ahead = value;
            return EDEN_OK;
        case EDEN_OPT_SLAB_MIB:
            if (value < 0 || value > 4096) return EDEN_ERR_INVALID_ARG;
            ctx->slab_mib = value;
            return EDEN_OK;
        case EDEN_OPT_SLAB_SIDES:
            if (value < 1 || value > 3) return EDEN_ERR_INVALID_ARG;
            ctx->slab_sides = value;
            return EDEN_OK;
        case EDEN_OPT_SLAB_STREAMS:
            if (value < 1 || value > 4) return EDEN_ERR_INVALID_ARG;
            ctx->slab_streams = value;
            return EDEN_OK;
        default:
            return EDEN_ERR_INVALID_ARG;
    }
}

extern "C" int eden_profile_enable(eden_ctx* ctx, int on)
{
    if (!ctx) return EDEN_ERR_INVALID_ARG;
    ctx->profiling = on != 0;
    ctx->records.clear();
    ctx->summary.clear();
    return EDEN_OK;
}

extern "C" int eden_profile_collect(eden_ctx* ctx, uint32_t* n_kernels)
{
    if (!ctx || !n_kernels) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
    ctx->summary.clear();
    for (const ProfileRecord& r : ctx->records) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) return EDEN_ERR_CUDA;
        ProfileSummary* s = nullptr;
        for (ProfileSummary& t : ctx->summary)
            if (std::strcmp(t.name, r.name) == 0) s = &t;
        if (!s) {
            ctx->summary.push_back(ProfileSummary{r.name, 0, 0.0, 0.0});
            s = &ctx->summary.back();
        }
        s->launches += 1;
        s->ms += ms;
        s->bytes += r.bytes;
    }
    ctx->records.clear();
    *n_kernels = (uint32_t)ctx->summary.size();
    return EDEN_OK;
}

extern "C" int eden_profile_get(eden_ctx* ctx, uint32_t i, const char** name, uint64_t* launches,
                                double* ms_total, double* bytes_total)
{
    if (!ctx || i >= ctx->summary.size() || !name || !launches || !ms_total || !bytes_total)
        return EDEN_ERR_INVALID_ARG;
    *name = ctx->summary[i].name;
    *launches = ctx->summary[i].launches;
    *ms_total = ctx->summary[i].ms;
    *bytes_total = ctx->summary[i].bytes;
    return EDEN_OK;
}

extern "C" int eden_status(eden_ctx* ctx, uint32_t* word)
{
    if (!ctx || !word) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    CUDA_OK(cudaMemcpyAsync(word, ctx->ws, sizeof(uint32_t), cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_OK(cudaMemsetAsync(ctx->ws, 0, sizeof(uint32_t), ctx->stream));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
    return EDEN_OK;
}

extern "C" int eden_client_stats(eden_ctx* ctx, uint32_t n, eden_client_stat* out)
{
    if (!ctx || !out || n != ctx->order.size()) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    std::vector<ClientState> st(n);
    CUDA_OK(cudaMemcpyAsync(st.data(), ctx->ws + ctx->states_off, n * sizeof(ClientState),
                            cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
    for (uint32_t j = 0; j < n; ++j) {
        eden_client_stat& o = out[ctx->order[j]];
        o.norm2 = st[j].norm2;
        o.dot = st[j].dot;
        o.received = st[j].received;
        o.flags = st[j].flags;
        o.reserved = 0;
    }
    return EDEN_OK;
}

// ------------------------------------------------------------------------------------
// planning
// ------------------------------------------------------------------------------------
namespace {

struct ClientPlan {
    uint32_t index;      // position in the caller's arrays
    uint64_t k, D;
    int L, W;
    bool subbit;
    bool needs_work;
    uint32_t coin_thr;   // non-integer b > 1
    double delta;        // uniform-interval family (Section 4.3): interval width; else 0
};

// A set of clients of one rotation dimension launched together.
struct Group {
    std::vector<uint32_t> members;   // indices into the plan array
    int L;
    bool subbit;
    bool fractional;                 // non-integer budgets b > 1
    bool uniform;                    // uniform-interval family: one signed byte per coordinate
};

struct CallLayout {
    uint64_t descs_off, states_off, utab_off, work_off, work_bytes;
};

constexpr uint64_t kUniformTableBytes = kUniformValues * sizeof(float);

// `delta` non-null: every client uses the uniform-interval family of that width (then
// `bits` is not read): one byte per rotated coordinate, no sparsification.
int plan_clients(uint64_t d, uint32_t n, const double* bits, const double* delta, std::vector<ClientPlan>& plan)
{
    if (d == 0 || n == 0 || (!bits && !delta)) return EDEN_ERR_INVALID_ARG;
    if (d > EDEN_MAX_DIM) return EDEN_ERR_TOO_LARGE;
    plan.resize(n);
    for (uint32_t c = 0; c < n && delta; ++c) {
        if (!(delta[c] >= kUniformMinDelta) || !(delta[c] < kUniformMaxDelta)) return EDEN_ERR_UNSUPPORTED_BITS;
        ClientPlan& p = plan[c];
        p.index = c;
        p.k = d;
        p.D = eden_rot_dim(d, 1.0);
        p.L = ceil_log2(p.D);
        p.W = 8;
        p.subbit = false;
        p.coin_thr = 0;
        p.delta = delta[c];
        p.needs_work = p.L > kGenericTileLog;
    }
    for (uint32_t c = 0; c < n && !delta; ++c) {
        const uint32_t W = eden_code_width(bits[c]);
        if (W == 0) return EDEN_ERR_UNSUPPORTED_BITS;
        ClientPlan& p = plan[c];
        p.index = c;
        p.k = eden_kept_count(d, bits[c]);
        p.D = eden_rot_dim(d, bits[c]);
        p.L = ceil_log2(p.D);
        p.W = (int)W;
        p.subbit = bits[c] < 1.0;
        p.coin_thr = coin_threshold(bits[c]);
        p.delta = 0.0;
        p.needs_work = p.subbit || p.L > kGenericTileLog;
    }
    return EDEN_OK;
}

int carve(const eden_ctx* ctx, uint64_t d, uint32_t n, bool uniform, CallLayout& lay)
{
    const FixedLayout f = fixed_layout(d);
    lay.descs_off = f.end;
    lay.states_off = lay.descs_off + align_up(sizeof(ClientDesc) * (uint64_t)n, 256);
    lay.utab_off = lay.states_off + align_up(sizeof(ClientState) * (uint64_t)n, 256);
    lay.work_off = lay.utab_off + (uniform ? kUniformTableBytes * (uint64_t)n : 0);
    if (lay.work_off > ctx->ws_bytes) return EDEN_ERR_WORKSPACE;
    lay.work_bytes = ctx->ws_bytes - lay.work_off;
    return EDEN_OK;
}

// One client's intermediate vector in the workspace; what follows it stays 256-byte aligned.
uint64_t work_buffer_bytes(uint64_t D) { return align_up(D * sizeof(float), 256); }

constexpr uint64_t kBatchHistBytes = 3ull * kSelBins * sizeof(uint32_t);

// Scratch of the exact-size mask selection for one client with b < 1.
constexpr uint64_t kCandBytes = (uint64_t)kSelCandCap * sizeof(uint2);

// The two-pass selection holds the keys that share tau's first digit, about d / 2048 of
// them (a binomial count): used while that, with a margin of many standard deviations,
// fits the candidate list.
bool two_pass_selection(const eden_ctx* ctx, uint64_t d)
{
    if (ctx->sel_rounds == 3) return false;      // EDEN_OPT_SEL_ROUNDS: three rounds at every size
    const double mean = (double)d / (double)kSelBins;
    return mean + 12.0 * std::sqrt(mean) + 64.0 <= (double)kSelCandCap;
}

// One-pass selection: the keys are independent uniform 32-bit words, so the k-th smallest
// of d lies near (k/d)*2^32 with a standard deviation of sqrt(p(1-p)/d)*2^32.  The band is
// that centre plus or minus `tenths`/10 standard deviations, narrowed where the keys it is
// expected to hold would not fit the candidate list; below three standard deviations the
// prediction is not worth a pass and the band is left empty (lo > hi), which sends the job
// to the histogram round.  A wrong prediction costs time, never the result.
void predicted_band(uint64_t d, uint64_t k, int tenths, uint32_t* lo, uint32_t* hi)
{
    *lo = 1u;
    *hi = 0u;
    if (d == 0 || k == 0 || k > d || tenths <= 0) return;
    const double two32 = 4294967296.0;
    const double p = (double)k / (double)d;
    const double sd = std::sqrt(p * (1.0 - p) / (double)d) * two32;
    double half = 0.1 * tenths * sd + 2.0;
    // expected candidates d * (2 half + 1) / 2^32, kept six of its own deviations under the cap
    const double room = (double)kSelCandCap - 6.0 * std::sqrt((double)kSelCandCap) - 64.0;
    const double half_max = (room * two32 / (double)d - 1.0) / 2.0;
    if (half > half_max) {
        half = half_max;
        if (half < 3.0 * sd) return;
    }
    const double centre = p * two32;
    const double a = std::floor(centre - half), b = std::ceil(centre + half);
    *lo = a < 0.0 ? 0u : (uint32_t)a;
    *hi = b > two32 - 1.0 ? 0xFFFFFFFFu : (uint32_t)b;
}

// mask bitmap of one job: 32 words per chunk of 1024 coordinates
uint64_t keep_bitmap_bytes(uint64_t d)
{
    return align_up((d + kSelChunk - 1) / kSelChunk * (kSelChunk / 8), 256);
}

uint64_t sel_scratch_bytes(const eden_ctx* ctx, uint64_t d)
{
    const uint64_t n_chunks = (d + kSelChunk - 1) / kSelChunk;
    return 256 + kBatchHistBytes + align_up(n_chunks * sizeof(unsigned long long), 256) +
           align_up(sizeof(SelJob), 256) + (two_pass_selection(ctx, d) ? kCandBytes + keep_bitmap_bytes(d) : 0);
}

// Groups: clients of one rotation dimension (and, within it, of one kind: b >= 1 or
// b < 1) are launched together, split so that each group's work buffers and selection
// scratch fit the workspace.  Larger dimensions first, so that for the mean a group with
// b >= 1, which covers every output coordinate, comes before any b < 1 group.
// `scratch_outside`: the selection scratch of the b < 1 clients lives elsewhere (SelectionAhead).
int make_groups(const eden_ctx* ctx, const std::vector<ClientPlan>& plan, uint64_t d, uint64_t work_bytes,
                std::vector<Group>& groups, bool scratch_outside = false)
{
    std::vector<uint32_t> idx(plan.size());
    for (uint32_t c = 0; c < plan.size(); ++c) idx[c] = c;
    std::stable_sort(idx.begin(), idx.end(), [&](uint32_t a, uint32_t b) {
        if (plan[a].subbit != plan[b].subbit) return !plan[a].subbit;
        if (plan[a].L != plan[b].L) return plan[a].L > plan[b].L;
        if ((plan[a].coin_thr != 0) != (plan[b].coin_thr != 0)) return plan[a].coin_thr == 0;
        return plan[a].W < plan[b].W;
    });
    size_t i = 0;
    while (i < idx.size()) {
        Group g;
        g.L = plan[idx[i]].L;
        g.subbit = plan[idx[i]].subbit;
        g.fractional = plan[idx[i]].coin_thr != 0;
        g.uniform = plan[idx[i]].delta > 0.0;
        const uint64_t need = (plan[idx[i]].needs_work ? work_buffer_bytes(plan[idx[i]].D) : 0) +
                              (g.subbit && !scratch_outside ? sel_scratch_bytes(ctx, d) : 0);
        if (need > work_bytes) return EDEN_ERR_WORKSPACE;
        uint64_t used = 0;
        while (i < idx.size() && plan[idx[i]].L == g.L && plan[idx[i]].subbit == g.subbit &&
               (plan[idx[i]].coin_thr != 0) == g.fractional &&
               used + need <= work_bytes && g.members.size() < 32768) {
            g.members.push_back(idx[i]);
            used += need;
            ++i;
        }
        groups.push_back(g);
    }
    return EDEN_OK;
}

// Mean code width of a group's members (bits per rotated coordinate on the wire).
double code_bits_per_coord(const std::vector<ClientPlan>& plan, const Group& g)
{
    double w = 0.0;
    for (uint32_t m : g.members) w += plan[m].W;
    return w / (double)g.members.size();
}

// Column passes over the bits above the row pass, top range first.
struct BitRange { int lo, lr; };

void column_ranges(int L, int lc, int max_lr, std::vector<BitRange>& out)
{
    const int rem = L - lc;
    if (rem <= 0) return;
    const int passes = (rem + max_lr - 1) / max_lr;
    int hi = L;
    for (int p = 0; p < passes; ++p) {
        const int lr = (hi - lc + (passes - p) - 1) / (passes - p);
        out.push_back({hi - lr, lr});
        hi -= lr;
    }
}

PassGeom column_geom(const BitRange& r)
{
    PassGeom g;
    g.lr = r.lr;
    g.lo = r.lo;
    g.lw = std::min(r.lo, kGenericTileLog - r.lr);
    g.lt = g.lw + g.lr;
    return g;
}

PassGeom row_geom(int lc) { return PassGeom{lc, lc, lc, 0}; }

// Plan of the register-blocked path.  The row pass covers index bits [0, 13 + row_lc);
// each column pass covers bits [lo, lo + lr + lc), lr of them inside a block and lc (0 or
// 3) across the 8 blocks of a cluster.  variant 0 (the default) uses no clusters; 1..3 are
// the cluster plans (two sweeps over HBM up to 2^27 coordinates), kept for tuning.
struct FastPass { int lo, lr, lc; };
struct FastPlan { int row_lc; std::vector<FastPass> cols; };   // cols: top range first

FastPlan fast_plan(int L, int variant)
{
    FastPlan pl;
    const int cb = L - kFastTileLog;
    if (variant == 0 || cb <= kFastMaxColBits) {
        // No clusters.  The pass that touches the fp32 vectors (the sender's first, the
        // receiver's last) also flips signs, takes the norm or loops over clients, so it
        // gets the fewest bits; the in-place middle passes run at copy speed for any
        // width up to 8 and take 8 bits each (measured: cfg4 648 -> 666 GB/s, cfg5
        // 423 -> 440 GB/s against an even split).  Measured on B200 this also beats every
        // cluster plan below: one more sweep over HBM costs less than the per-tile
        // cluster barriers.
        pl.row_lc = 0;
        const int passes = (cb + kFastMaxColBits - 1) / kFastMaxColBits;
        const int top = cb - kFastMaxColBits * (passes - 1);
        int hi = L;
        for (int p = 0; p < passes; ++p) {
            const int bits = p == 0 ? top : kFastMaxColBits;
            pl.cols.push_back(FastPass{hi - bits, bits, 0});
            hi -= bits;
        }
        return pl;
    }
    auto one = [](int lo, int bits) {
        return bits > kFastMaxColBits ? FastPass{lo, bits - kFastClusterLog, kFastClusterLog}
                                      : FastPass{lo, bits, 0};
    };
    if (cb <= kFastMaxColBits + kFastClusterLog && variant != 3) {
        if (variant == 1) {            // cluster on the column pass
            pl.row_lc = 0;
            pl.cols.push_back(FastPass{kFastTileLog, cb - kFastClusterLog, kFastClusterLog});
        } else {                       // variant 2: cluster on the row pass
            pl.row_lc = kFastClusterLog;
            pl.cols.push_back(FastPass{kFastTileLog + kFastClusterLog, cb - kFastClusterLog, 0});
        }
    } else {                           // clusters on both (variant 3, or more than 11 bits)
        pl.row_lc = kFastClusterLog;
        const int low = kFastTileLog + kFastClusterLog;
        const int rest = L - low;
        const int per = kFastMaxColBits + kFastClusterLog;
        const int passes = (rest + per - 1) / per;
        int hi = L;
        for (int p = 0; p < passes; ++p) {
            const int bits = (hi - low + (passes - p) - 1) / (passes - p);
            pl.cols.push_back(one(hi - bits, bits));
            hi -= bits;
        }
    }
    return pl;
}

// launch with a thread-block cluster of 2^lc blocks along x (lc = 0: ordinary launch)
template <typename... KArgs, typename... Args>
cudaError_t launch_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, int lc, cudaStream_t stream,
                           Args... args)
{
    cudaLaunchConfig_t cfg;
    std::memset(&cfg, 0, sizeof(cfg));
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1u << lc;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = lc > 0 ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

#define LAUNCH_CL(ctx, name, bytes, kernel, grid, block, lc, ...)                            \
    do {                                                                                     \
        profile_begin(ctx, name, (double)(bytes));                                           \
        const cudaError_t e_ = launch_cluster(kernel, grid, block, lc, (ctx)->stream, __VA_ARGS__); \
        profile_end(ctx);                                                                    \
        ++(ctx)->launches;                                                                   \
        if (e_ != cudaSuccess || cudaGetLastError() != cudaSuccess) return EDEN_ERR_CUDA;    \
    } while (0)

#define EDEN_DISPATCH_LR(lr, CALL)                \
    switch (lr) {                                 \
        case 1: { constexpr int LR_ = 1; CALL; } break; \
        case 2: { constexpr int LR_ = 2; CALL; } break; \
        case 3: { constexpr int LR_ = 3; CALL; } break; \
        case 4: { constexpr int LR_ = 4; CALL; } break; \
        case 5: { constexpr int LR_ = 5; CALL; } break; \
        case 6: { constexpr int LR_ = 6; CALL; } break; \
        case 7: { constexpr int LR_ = 7; CALL; } break; \
        case 8: { constexpr int LR_ = 8; CALL; } break; \
        default: return EDEN_ERR_INVALID_ARG;     \
    }

#define EDEN_DISPATCH_LC(lc, CALL)                \
    switch (lc) {                                 \
        case 0: { constexpr int LC_ = 0; CALL; } break; \
        case 3: { constexpr int LC_ = 3; CALL; } break; \
        default: return EDEN_ERR_INVALID_ARG;     \
    }

#define EDEN_DISPATCH_FRAC(frac, CALL)            \
    if (frac) { constexpr bool FRAC_ = true; CALL; } else { constexpr bool FRAC_ = false; CALL; }

#define EDEN_DISPATCH_W(w, CALL)                  \
    switch (w) {                                  \
        case 1: { constexpr int W_ = 1; CALL; } break; \
        case 2: { constexpr int W_ = 2; CALL; } break; \
        case 3: { constexpr int W_ = 3; CALL; } break; \
        case 4: { constexpr int W_ = 4; CALL; } break; \
        case 5: { constexpr int W_ = 5; CALL; } break; \
        case 6: { constexpr int W_ = 6; CALL; } break; \
        case 7: { constexpr int W_ = 7; CALL; } break; \
        case 8: { constexpr int W_ = 8; CALL; } break; \
        default: return EDEN_ERR_INVALID_ARG;     \
    }

// Runs of equal code width inside a group (members are sorted by width within a group).
struct WidthRun { uint32_t first, count; int W; };

void width_runs(const std::vector<ClientPlan>& plan, const Group& g, std::vector<WidthRun>& runs)
{
    for (uint32_t j = 0; j < g.members.size(); ++j) {
        const int W = plan[g.members[j]].W;
        if (!runs.empty() && runs.back().W == W) ++runs.back().count;
        else runs.push_back({j, 1u, W});
    }
}

// Blocks of `kernel` that fit on the device at once (cached per kernel and device).
template <typename K>
int resident_blocks(const eden_ctx* ctx, K kernel, uint32_t dynamic_smem)
{
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, int> cache;
    std::lock_guard<std::mutex> lock(mu);
    const auto key = std::make_pair((const void*)kernel, ctx->device);
    auto it = cache.find(key);
    if (it != cache.end()) return it->second;
    int per_sm = 0;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dynamic_smem) != cudaSuccess)
        return -1;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kFastThreads, dynamic_smem) != cudaSuccess ||
        per_sm < 1)
        return -1;
    return cache[key] = per_sm * ctx->sm_count;
}

// Slab order on several streams: the slabs are independent, so they are dealt round-robin
// to side streams that fork from the context's stream and join it again; the launch macros
// follow ctx->stream, which SlabStreams points at the stream of the current slab.
struct SlabStreams {
    eden_ctx* ctx;
    cudaStream_t main;
    int n;
    bool ok;
    explicit SlabStreams(eden_ctx* c) : ctx(c), main(c->stream), n(c->slab_streams), ok(true)
    {
        if (n <= 1) return;
        while ((int)ctx->side.size() < n && ok) {
            cudaStream_t st;
            ok = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking) == cudaSuccess;
            if (ok) ctx->side.push_back(st);
        }
        while (ctx->slab_events.size() < (size_t)n + 1 && ok) {
            cudaEvent_t e;
            ok = cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
            if (ok) ctx->slab_events.push_back(e);
        }
        if (!ok) return;
        ok = cudaEventRecord(ctx->slab_events[0], main) == cudaSuccess;
        for (int j = 0; j < n && ok; ++j) ok = cudaStreamWaitEvent(ctx->side[j], ctx->slab_events[0], 0) == cudaSuccess;
    }
    void use(unsigned slab) { if (n > 1 && ok) ctx->stream = ctx->side[slab % (unsigned)n]; }
    ~SlabStreams()
    {
        ctx->stream = main;
        if (n <= 1 || !ok) return;
        for (int j = 0; j < n; ++j) {
            cudaEventRecord(ctx->slab_events[1 + j], ctx->side[j]);
            cudaStreamWaitEvent(main, ctx->slab_events[1 + j], 0);
        }
    }
};

// Sender passes of one group on the register-blocked path.
// `h_descs`: the host copy of the group's descriptors (d_descs is the same array on the device).
// `fold_scales`: small rounds: the row pass writes the scales itself (no k_enc_scale); else nullptr.
int fast_encode_group(eden_ctx* ctx, const std::vector<ClientPlan>& plan, const Group& g, const ClientDesc* h_descs,
                      ClientDesc* d_descs, ClientState* d_states, uint64_t d, uint32_t* d_status, float* fold_scales)
{
    const uint32_t gn = (uint32_t)g.members.size();
    const double D = (double)(1ull << g.L);
    const unsigned tiles = (unsigned)((1ull << g.L) >> kFastTileLog);
    // the uniform-interval family has no cluster form of the row pass
    const FastPlan pl = fast_plan(g.L, g.uniform ? 0 : ctx->plan_variant);
    // Slab order (EDEN_OPT_SLAB_MIB, three-sweep plans without clusters): after the top pass
    // the sub-vectors of 2^(13 + middle bits) coordinates are independent, so the middle and
    // the row pass can run slab by slab (some sub-vectors of some clients at a time), the row
    // pass reading what the middle pass has just written while it may still be in L2.
    const bool slabs = ctx->slab_mib > 0 && (ctx->slab_sides & 1) && pl.cols.size() == 2 && pl.row_lc == 0 &&
                       pl.cols[0].lc == 0 && pl.cols[1].lc == 0 && !g.uniform && !ctx->row_staging;
    std::vector<WidthRun> runs;
    width_runs(plan, g, runs);
    for (const WidthRun& r : runs)
        // the row pass addresses client j of the run at work0 + j * 2^L
        for (uint32_t j = 0; j < r.count; ++j)
            if (h_descs[r.first + j].work != h_descs[r.first].work + ((uint64_t)j << g.L)) return EDEN_ERR_INVALID_ARG;
    for (size_t pi = 0; pi < pl.cols.size(); ++pi) {
        const FastPass& ps = pl.cols[pi];
        if (pi == 0) {
            EDEN_DISPATCH_LC(ps.lc, EDEN_DISPATCH_LR(ps.lr,
                LAUNCH_CL(ctx, "f_enc_first", gn * (4.0 * std::min<double>((double)d, D) + 4.0 * D),
                          (k_f_col<LR_, LC_, true>), dim3(tiles, gn), dim3(kFastThreads), ps.lc,
                          (const ClientDesc*)d_descs, d_states, ps.lo, 0, 0u)));
        } else if (!slabs) {
            EDEN_DISPATCH_LC(ps.lc, EDEN_DISPATCH_LR(ps.lr,
                LAUNCH_CL(ctx, "f_mid", gn * 8.0 * D, (k_f_col<LR_, LC_, false>), dim3(tiles, gn),
                          dim3(kFastThreads), ps.lc, (const ClientDesc*)d_descs, d_states, ps.lo, 1, 0u)));
        }
    }
    const int inv_ready = pl.cols.size() >= 2 ? 1 : 0;     // a middle pass has left 1/||y|| in the client's state
    if (slabs) {
        const FastPass& ps = pl.cols[1];
        const unsigned sub_tiles = 1u << ps.lr;                         // tiles of one independent sub-vector
        const uint64_t sub_mib = ((uint64_t)sub_tiles << kFastTileLog) * 4 >> 20;
        SlabStreams fork(ctx);
        if (!fork.ok) return EDEN_ERR_CUDA;
        unsigned slab = 0;
        for (const WidthRun& r : runs) {
            const uint32_t cl = (uint32_t)std::min<uint64_t>(r.count, std::max<uint64_t>(1, ctx->slab_mib / std::max<uint64_t>(1, sub_mib)));
            const unsigned subs = (unsigned)std::max<uint64_t>(1, ctx->slab_mib / std::max<uint64_t>(1, sub_mib * cl));
            for (uint32_t c0 = 0; c0 < r.count; c0 += cl) {
                const uint32_t cn = std::min(cl, r.count - c0);
                const ClientDesc* dd = d_descs + r.first + c0;
                ClientState* ds = d_states + r.first + c0;
                for (unsigned t0 = 0; t0 < tiles; t0 += subs * sub_tiles) {
                    const unsigned tn = std::min(subs * sub_tiles, tiles - t0);
                    fork.use(slab++);
                    EDEN_DISPATCH_LR(ps.lr,
                        LAUNCH_CL(ctx, "f_mid", cn * 8.0 * 8192.0 * tn, (k_f_col<LR_, 0, false>), dim3(tn, cn),
                                  dim3(kFastThreads), 0, dd, ds, ps.lo, 1, t0));
                    EDEN_DISPATCH_FRAC(g.fractional, EDEN_DISPATCH_W(r.W,
                        LAUNCH_CL(ctx, "f_enc_last", cn * (4.0 + r.W / 8.0) * 8192.0 * tn, (k_f_enc_last<W_, 0, FRAC_>),
                                  dim3(tn, cn), dim3(kFastThreads), 0, dd, ds,
                                  (const float*)h_descs[r.first + c0].work, g.L, inv_ready, t0, fold_scales, d_status)));
                }
            }
        }
        return EDEN_OK;
    }
    for (const WidthRun& r : runs) {
        if (g.uniform) {
            LAUNCH(ctx, "f_enc_last", r.count * 5.0 * D, (k_f_enc_last<8, 0, false, true>), dim3(tiles, r.count),
                   kFastThreads, 0, (const ClientDesc*)(d_descs + r.first), d_states + r.first,
                   (const float*)h_descs[r.first].work, g.L, inv_ready, 0u, fold_scales, d_status);
            continue;
        }
        if (ctx->row_staging && pl.row_lc == 0) {
            const int tiles_log = g.L - kFastTileLog;
            const uint32_t total = r.count << tiles_log;
            EDEN_DISPATCH_FRAC(g.fractional, EDEN_DISPATCH_W(r.W, {
                const int resident = resident_blocks(ctx, k_f_enc_last_staged<W_, FRAC_>, kStagedDynamicBytes);
                if (resident < 1) return EDEN_ERR_CUDA;
                const uint32_t blocks = std::min<uint32_t>(total, (uint32_t)resident);
                LAUNCH(ctx, "f_enc_last", r.count * (4.0 + r.W / 8.0) * D, (k_f_enc_last_staged<W_, FRAC_>),
                       blocks, kFastThreads, kStagedDynamicBytes, (const ClientDesc*)(d_descs + r.first), d_states + r.first,
                       total, tiles_log, d_status);
            }));
            continue;
        }
        EDEN_DISPATCH_FRAC(g.fractional, EDEN_DISPATCH_LC(pl.row_lc, EDEN_DISPATCH_W(r.W,
            LAUNCH_CL(ctx, "f_enc_last", r.count * (4.0 + r.W / 8.0) * D, (k_f_enc_last<W_, LC_, FRAC_>),
                      dim3(tiles, r.count), dim3(kFastThreads), pl.row_lc,
                      (const ClientDesc*)(d_descs + r.first), d_states + r.first,
                      (const float*)h_descs[r.first].work, g.L, inv_ready, 0u, fold_scales, d_status))));
    }
    return EDEN_OK;
}

// Receiver passes of one group on the register-blocked path.
// `part`/`part_bytes`: free workspace behind the group's work buffers, for partial sums.
// `fold_scales`: small rounds: the row pass does k_dec_prep's work from these scales; else nullptr.
int fast_decode_group(eden_ctx* ctx, const std::vector<ClientPlan>& plan, const Group& g,
                      ClientDesc* d_descs, ClientState* d_states, float* out, uint64_t d, int mode,
                      float* part, uint64_t part_bytes, const float* fold_scales, uint32_t* d_status)
{
    ClientState* const fold_states = fold_scales ? d_states : nullptr;
    const uint32_t gn = (uint32_t)g.members.size();
    const double D = (double)(1ull << g.L);
    const unsigned tiles = (unsigned)((1ull << g.L) >> kFastTileLog);
    const FastPlan pl = fast_plan(g.L, ctx->plan_variant);
    std::vector<WidthRun> runs;
    width_runs(plan, g, runs);
    // slab order as on the sender (EDEN_OPT_SLAB_MIB): row pass, then middle pass, slab by slab
    const bool slabs = ctx->slab_mib > 0 && (ctx->slab_sides & 2) && pl.cols.size() == 2 && pl.row_lc == 0 &&
                       pl.cols[0].lc == 0 && pl.cols[1].lc == 0;
    if (slabs) {
        const FastPass& ps = pl.cols[1];
        const unsigned sub_tiles = 1u << ps.lr;
        const uint64_t sub_mib = ((uint64_t)sub_tiles << kFastTileLog) * 4 >> 20;
        SlabStreams fork(ctx);
        if (!fork.ok) return EDEN_ERR_CUDA;
        unsigned slab = 0;
        for (const WidthRun& r : runs) {
            const uint32_t cl = (uint32_t)std::min<uint64_t>(r.count, std::max<uint64_t>(1, ctx->slab_mib / std::max<uint64_t>(1, sub_mib)));
            const unsigned subs = (unsigned)std::max<uint64_t>(1, ctx->slab_mib / std::max<uint64_t>(1, sub_mib * cl));
            for (uint32_t c0 = 0; c0 < r.count; c0 += cl) {
                const uint32_t cn = std::min(cl, r.count - c0);
                const ClientDesc* dd = d_descs + r.first + c0;
                for (unsigned t0 = 0; t0 < tiles; t0 += subs * sub_tiles) {
                    const unsigned tn = std::min(subs * sub_tiles, tiles - t0);
                    fork.use(slab++);
                    EDEN_DISPATCH_FRAC(g.fractional, EDEN_DISPATCH_W(r.W,
                        LAUNCH_CL(ctx, "f_dec_first", cn * (4.0 + r.W / 8.0) * 8192.0 * tn, (k_f_dec_first<W_, 0, FRAC_>),
                                  dim3(tn, cn), dim3(kFastThreads), 0, dd, t0,
                                  fold_states ? fold_states + r.first + c0 : nullptr, fold_scales, d_status)));
                    EDEN_DISPATCH_LR(ps.lr,
                        LAUNCH_CL(ctx, "f_mid", cn * 8.0 * 8192.0 * tn, (k_f_col<LR_, 0, false>), dim3(tn, cn),
                                  dim3(kFastThreads), 0, dd, d_states + r.first + c0, ps.lo, 0, t0));
                }
            }
        }
    } else {
        for (const WidthRun& r : runs) {
            EDEN_DISPATCH_FRAC(g.fractional, EDEN_DISPATCH_LC(pl.row_lc, EDEN_DISPATCH_W(r.W,
                LAUNCH_CL(ctx, "f_dec_first", r.count * (4.0 + r.W / 8.0) * D, (k_f_dec_first<W_, LC_, FRAC_>),
                          dim3(tiles, r.count), dim3(kFastThreads), pl.row_lc,
                          (const ClientDesc*)(d_descs + r.first), 0u,
                          fold_states ? fold_states + r.first : nullptr, fold_scales, d_status))));
        }
    }
    // the receiver walks the column ranges bottom-up so that the top range comes last
    for (size_t pi = pl.cols.size(); pi-- > 0;) {
        const FastPass& ps = pl.cols[pi];
        if (pi > 0) {
            if (slabs) continue;
            EDEN_DISPATCH_LC(ps.lc, EDEN_DISPATCH_LR(ps.lr,
                LAUNCH_CL(ctx, "f_mid", gn * 8.0 * D, (k_f_col<LR_, LC_, false>), dim3(tiles, gn),
                          dim3(kFastThreads), ps.lc, (const ClientDesc*)d_descs, d_states, ps.lo, 0, 0u)));
        } else {
            // A round with few tiles leaves most SMs idle if every block walks all clients:
            // split the clients over block rows, each row summing into a partial vector of
            // its own, and add the partial vectors up afterwards (a fixed order, so the
            // result does not depend on scheduling).
            const uint64_t stride = align_up(d, 64);
            uint32_t rows = 1, per = gn;
            if (mode != OUT_YHAT && ps.lc == 0 && gn >= 2 && tiles < 2u * (unsigned)ctx->sm_count) {
                const uint32_t want = std::min<uint32_t>(std::min<uint32_t>(gn, 16u),
                                                         (2u * (unsigned)ctx->sm_count + tiles - 1) / tiles);
                per = (gn + want - 1) / want;
                rows = (gn + per - 1) / per;
                if (rows < 2 || (uint64_t)rows * stride * sizeof(float) > part_bytes) { rows = 1; per = gn; }
            }
            if (rows > 1) {
                EDEN_DISPATCH_LR(ps.lr,
                    LAUNCH_CL(ctx, "f_dec_last", gn * 4.0 * D + rows * 4.0 * std::min<double>((double)d, D),
                              (k_f_dec_last<LR_, 0>), dim3(tiles, rows), dim3(kFastThreads), 0,
                              (const ClientDesc*)d_descs, (const ClientState*)d_states, per,
                              ps.lo, part, d, (int)OUT_PART, gn, stride));
                LAUNCH(ctx, "dec_sum", (rows + (mode == OUT_ACC ? 2.0 : 1.0)) * 4.0 * (double)d, k_sum_partials,
                       (unsigned)((d + 1023) / 1024), 256, 0, (const float*)part, rows, stride, d, out,
                       mode == OUT_ACC ? 1 : 0);
            } else {
                EDEN_DISPATCH_LC(ps.lc, EDEN_DISPATCH_LR(ps.lr,
                    LAUNCH_CL(ctx, "f_dec_last",
                              gn * 4.0 * D + (mode == OUT_ACC ? 8.0 : 4.0) * std::min<double>((double)d, D),
                              (k_f_dec_last<LR_, LC_>), dim3(tiles, mode == OUT_YHAT ? gn : 1u), dim3(kFastThreads), ps.lc,
                              (const ClientDesc*)d_descs, (const ClientState*)d_states, mode == OUT_YHAT ? 1u : gn,
                              ps.lo, out, d, mode, gn, (uint64_t)0)));
            }
        }
    }
    return EDEN_OK;
}

// rounds of at most this many row-pass tiles (2^25 coordinates) fold their small kernels into the row pass
// (at 2^28 the fence per tile already costs the sender's row pass 7 %)
constexpr uint64_t kFoldMaxTiles = 4096;
constexpr uint64_t kFoldMaxMaskWords = 256;    // ... if a client's received-bitmap is at most this long

bool fast_eligible(const eden_ctx* ctx, const Group& g)
{
    return !ctx->force_generic && g.L > kFastTileLog && g.L <= 40;
}

// Exact-size mask selection for one client (Section 4.1): fills the MaskSelect and the
// scanned chunk offsets in the fixed scratch.
int run_selection(eden_ctx* ctx, const FixedLayout& f, uint64_t seed, uint64_t d, uint64_t k)
{
    MaskSelect* sel = (MaskSelect*)(ctx->ws + f.sel);
    uint32_t* hist = (uint32_t*)(ctx->ws + f.hist);
    unsigned long long* chunks = (unsigned long long*)(ctx->ws + f.chunks);
    const uint64_t calls = (d + 3) / 4;
    const unsigned grid = (unsigned)((calls + kSelThreads - 1) / kSelThreads);
    CUDA_OK(cudaMemsetAsync(hist, 0, kHistBytes, ctx->stream));
    LAUNCH(ctx, "sel_hist", 0, k_sel_hist, grid, kSelThreads, 0, seed, d, 0, sel, hist);
    LAUNCH(ctx, "sel_find", 65536 * 4, k_sel_find, 1, 1024, 0, hist, k, 0, sel);
    LAUNCH(ctx, "sel_hist", 0, k_sel_hist, grid, kSelThreads, 0, seed, d, 1, sel, hist + 65536);
    LAUNCH(ctx, "sel_find", 65536 * 4, k_sel_find, 1, 1024, 0, hist + 65536, k, 1, sel);
    LAUNCH(ctx, "sel_chunk_count", grid * 8.0, k_sel_chunk_count, grid, kSelThreads, 0, seed, d, sel, chunks);
    LAUNCH(ctx, "sel_chunk_scan", grid * 16.0, k_sel_chunk_scan, 1, 1024, 0, chunks, (uint64_t)grid);
    return EDEN_OK;
}

}  // namespace

namespace {

// Selection jobs of a group of clients with b < 1.  The scratch sits behind the group's
// work buffers, or in the arena of a call that selects ahead (SelectionAhead): n MaskSelect
// slots, n histogram triples (contiguous with the slots, cleared by one memset), n chunk
// arrays, the job table itself, then the candidate lists and the mask bitmaps.
struct SelBatch {
    SelJob* d_jobs;
    uint32_t n;
    unsigned grid;       // blocks of 1024 coordinates
    bool two_pass;       // the jobs carry mask bitmaps (k_selc_compact / k_selc_scatter)
    std::vector<const uint32_t*> keep;   // two_pass: device address of each job's bitmap
};

int start_selection_batch(eden_ctx* ctx, char* region, uint64_t d, const std::vector<SelJob>& partial,
                          SelBatch& batch)
{
    const uint32_t n = (uint32_t)partial.size();
    const uint64_t n_chunks = (d + kSelChunk - 1) / kSelChunk;
    const uint64_t chunk_bytes = align_up(n_chunks * sizeof(unsigned long long), 256);
    char* sel_base = region;
    char* hist_base = sel_base + 256ull * n;
    char* chunk_base = hist_base + kBatchHistBytes * n;
    char* job_base = chunk_base + chunk_bytes * n;
    char* cand_base = job_base + align_up(sizeof(SelJob), 256) * n;
    const bool two_pass = two_pass_selection(ctx, d);
    std::vector<SelJob> jobs(partial);
    for (uint32_t j = 0; j < n; ++j) {
        jobs[j].sel = (MaskSelect*)(sel_base + 256ull * j);
        jobs[j].hist = (uint32_t*)(hist_base + kBatchHistBytes * j);
        jobs[j].chunks = (unsigned long long*)(chunk_base + chunk_bytes * j);
        jobs[j].cand = two_pass ? (uint2*)(cand_base + kCandBytes * j) : nullptr;
        jobs[j].keep = two_pass ? (uint32_t*)(cand_base + kCandBytes * n + keep_bitmap_bytes(d) * j) : nullptr;
    }
    batch.two_pass = two_pass;
    batch.keep.clear();
    for (uint32_t j = 0; j < n; ++j) batch.keep.push_back(jobs[j].keep);
    batch.d_jobs = (SelJob*)job_base;
    batch.n = n;
    batch.grid = (unsigned)(((d + 3) / 4 + kSelThreads - 1) / kSelThreads);
    const unsigned hist_grid = (unsigned)(((d + 3) / 4 + (uint64_t)kSelThreads * kSelCallsPerThread - 1) /
                                          ((uint64_t)kSelThreads * kSelCallsPerThread));
    const bool predict = two_pass && ctx->sel_rounds == 1;
    if (predict)
        for (uint32_t j = 0; j < n; ++j) predicted_band(jobs[j].d, jobs[j].k, ctx->sel_band, &jobs[j].lo, &jobs[j].hi);
    CUDA_OK(cudaMemcpyAsync(batch.d_jobs, jobs.data(), sizeof(SelJob) * n, cudaMemcpyHostToDevice, ctx->stream));
    // the MaskSelect slots (the fallback flags) and the histograms are contiguous
    CUDA_OK(cudaMemsetAsync(sel_base, 0, (256ull + kBatchHistBytes) * n, ctx->stream));
    const double keys = (double)n * (double)d;
    if (two_pass) {
        uint32_t* d_status = (uint32_t*)(ctx->ws + fixed_layout(1).status);
        const SelJob* dj = (const SelJob*)batch.d_jobs;
        const uint64_t n_chunks64 = batch.grid;
        const unsigned collect_grid = (batch.grid + kSelThreads / 32 - 1) / (kSelThreads / 32);
        if (predict) {
            // one pass over the keys; k_selc_redo only does the jobs whose threshold fell outside their band
            LAUNCH(ctx, "sel_collect", keys / 128.0, k_selc_collect<true>, dim3(collect_grid, n), kSelThreads, 0,
                   dj, n_chunks64);
            LAUNCH(ctx, "sel_resolve", keys / 64.0, k_selc_resolve<true>, n, 1024, 0, dj, d_status, n_chunks64);
            LAUNCH(ctx, "sel_redo", 0, k_selc_redo, n, 1024, 0, dj, d_status, n_chunks64);
            return EDEN_OK;
        }
        LAUNCH(ctx, "sel_hist", 0, k_selc_hist, dim3(hist_grid, n), kSelThreads, 0, dj);
        LAUNCH(ctx, "sel_find", n * (double)kSelBins * 4, k_selb_find, n, 1024, 0, dj, 0);
        LAUNCH(ctx, "sel_collect", keys / 128.0, k_selc_collect<false>, dim3(collect_grid, n), kSelThreads, 0,
               dj, n_chunks64);
        LAUNCH(ctx, "sel_resolve", keys / 64.0, k_selc_resolve<false>, n, 1024, 0, dj, d_status, n_chunks64);
        return EDEN_OK;
    }
    for (int round = 0; round < 3; ++round) {
        LAUNCH(ctx, "sel_hist", 0, k_selb_hist, dim3(hist_grid, n), kSelThreads, 0, (const SelJob*)batch.d_jobs, round);
        LAUNCH(ctx, "sel_find", n * (double)kSelBins * 4, k_selb_find, n, 1024, 0, (const SelJob*)batch.d_jobs, round);
    }
    LAUNCH(ctx, "sel_chunk_count", keys / 128.0, k_selb_chunk_count, dim3(batch.grid, n), kSelThreads, 0,
           (const SelJob*)batch.d_jobs);
    LAUNCH(ctx, "sel_chunk_scan", keys / 64.0, k_selb_chunk_scan, n, 1024, 0, (const SelJob*)batch.d_jobs,
           (uint64_t)batch.grid);
    return EDEN_OK;
}

// Selection ahead of its use.  The masks of a call's b < 1 clients depend on nothing but
// (seed, d, k), and finding them is integer arithmetic (the Philox keys) with next to no
// memory traffic, while the transform passes of the b >= 1 groups, which come first in the
// processing order, are bound by HBM.  So the selections of all b < 1 groups are enqueued on
// a side stream when the call starts, with their scratch in an arena at the end of the work
// region, and the main stream waits for a group's event only when it reaches that group.
// The launch macros follow ctx->stream, which begin() points at the side stream and end()
// puts back; the destructor joins the side stream into the main one whatever happened.
struct SelectionAhead {
    eden_ctx* ctx;
    cudaStream_t main;
    bool on, forked;
    uint64_t arena_off, arena_bytes;
    std::vector<SelBatch> batches;       // by group index (empty entries for b >= 1 groups)
    std::vector<int> event_of;           // by group index: its event in ctx->sel_events, -1 if none

    explicit SelectionAhead(eden_ctx* c) : ctx(c), main(c->stream), on(false), forked(false), arena_off(0), arena_bytes(0) {}

    // Decides whether this call selects ahead and shrinks the work region by the arena.
    void plan_arena(const std::vector<ClientPlan>& plan, uint64_t d, CallLayout& lay)
    {
        uint64_t n_sub = 0;
        for (const ClientPlan& p : plan) n_sub += p.subbit ? 1 : 0;
        if (!ctx->sel_ahead || n_sub == 0 || n_sub == plan.size()) return;
        const uint64_t bytes = n_sub * sel_scratch_bytes(ctx, d);
        if (bytes >= lay.work_bytes / 2) return;
        on = true;
        arena_bytes = bytes;
        lay.work_bytes -= bytes;
        arena_off = lay.work_off + lay.work_bytes;
    }
    void cancel(CallLayout& lay)
    {
        if (!on) return;
        on = false;
        lay.work_bytes += arena_bytes;
    }
    int begin(size_t n_groups)
    {
        batches.assign(n_groups, SelBatch{nullptr, 0, 0, false, {}});
        event_of.assign(n_groups, -1);
        if (!ctx->sel_stream && cudaStreamCreateWithFlags(&ctx->sel_stream, cudaStreamNonBlocking) != cudaSuccess) {
            ctx->sel_stream = nullptr;
            return EDEN_ERR_CUDA;
        }
        while (ctx->sel_events.size() < 2 + n_groups) {
            cudaEvent_t e;
            if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return EDEN_ERR_CUDA;
            ctx->sel_events.push_back(e);
        }
        // the arena may still be in use by earlier work on the main stream
        if (cudaEventRecord(ctx->sel_events[0], main) != cudaSuccess ||
            cudaStreamWaitEvent(ctx->sel_stream, ctx->sel_events[0], 0) != cudaSuccess)
            return EDEN_ERR_CUDA;
        forked = true;
        ctx->stream = ctx->sel_stream;
        return EDEN_OK;
    }
    // group gi's selection has been enqueued
    int mark(size_t gi)
    {
        event_of[gi] = (int)(2 + gi);
        return cudaEventRecord(ctx->sel_events[2 + gi], ctx->sel_stream) == cudaSuccess ? EDEN_OK : EDEN_ERR_CUDA;
    }
    void end() { ctx->stream = main; }
    // the main stream is about to use group gi's masks
    int wait(size_t gi)
    {
        if (event_of[gi] < 0) return EDEN_ERR_INVALID_ARG;
        return cudaStreamWaitEvent(main, ctx->sel_events[event_of[gi]], 0) == cudaSuccess ? EDEN_OK : EDEN_ERR_CUDA;
    }
    ~SelectionAhead()
    {
        ctx->stream = main;
        if (!forked) return;
        cudaEventRecord(ctx->sel_events[1], ctx->sel_stream);
        cudaStreamWaitEvent(main, ctx->sel_events[1], 0);
    }
};

}  // namespace

extern "C" int eden_mask_threshold_band(uint64_t d, uint64_t k, int tenths, uint32_t* lo, uint32_t* hi)
{
    if (!lo || !hi || d == 0 || k == 0 || k > d || tenths < 0 || tenths > 120) return EDEN_ERR_INVALID_ARG;
    predicted_band(d, k, tenths, lo, hi);
    return EDEN_OK;
}

// How one client's transform is split into sweeps over HBM (host only).
extern "C" int eden_pass_plan(uint64_t d, double bits, uint32_t* pass_bits, uint32_t max_passes,
                              uint32_t* n_passes)
{
    if (!pass_bits || !n_passes || d == 0 || d > EDEN_MAX_DIM || eden_code_width(bits) == 0)
        return EDEN_ERR_INVALID_ARG;
    const int L = ceil_log2(eden_rot_dim(d, bits));
    std::vector<uint32_t> out;
    if (L <= kGenericTileLog) {
        out.push_back((uint32_t)L);                       // one block per client
    } else {
        const FastPlan pl = fast_plan(L, 0);
        for (const FastPass& ps : pl.cols) out.push_back((uint32_t)(ps.lr + ps.lc));
        out.push_back((uint32_t)(kFastTileLog + pl.row_lc));
    }
    if (out.size() > max_passes) return EDEN_ERR_INVALID_ARG;
    std::copy(out.begin(), out.end(), pass_bits);
    *n_passes = (uint32_t)out.size();
    return EDEN_OK;
}

// ------------------------------------------------------------------------------------
// sender
// ------------------------------------------------------------------------------------
namespace {

// The call's descriptors and, right behind them in the workspace, its zeroed per-client
// state, in one copy (one stream operation less than a copy and a memset, which matters
// for small rounds).
int upload_descs_and_clear_states(eden_ctx* ctx, const CallLayout& lay, const std::vector<ClientDesc>& descs)
{
    const size_t n = descs.size();
    const size_t bytes = (size_t)(lay.states_off - lay.descs_off) + sizeof(ClientState) * n;
    std::vector<unsigned char> image(bytes, 0);
    std::memcpy(image.data(), descs.data(), sizeof(ClientDesc) * n);
    CUDA_OK(cudaMemcpyAsync(ctx->ws + lay.descs_off, image.data(), bytes, cudaMemcpyHostToDevice, ctx->stream));
    return EDEN_OK;
}

// Values of the uniform-interval family for the clients in processing order, uploaded
// behind the descriptors; sets each descriptor's table pointer and interval width.
int upload_uniform_tables(eden_ctx* ctx, const CallLayout& lay, const std::vector<ClientPlan>& plan,
                          const std::vector<uint32_t>& order, std::vector<ClientDesc>& descs)
{
    std::vector<float> tabs((size_t)kUniformValues * descs.size());
    std::map<double, size_t> seen;                 // clients usually share one width
    float* d_tabs = (float*)(ctx->ws + lay.utab_off);
    for (size_t j = 0; j < descs.size(); ++j) {
        const double delta = plan[order[j]].delta;
        auto it = seen.find(delta);
        if (it == seen.end()) {
            uniform_values(delta, &tabs[j * kUniformValues]);
            seen[delta] = j;
        } else {
            std::copy(&tabs[it->second * kUniformValues], &tabs[(it->second + 1) * kUniformValues],
                      &tabs[j * kUniformValues]);
        }
        descs[j].utable = d_tabs + j * kUniformValues;
        descs[j].delta = (float)delta;
    }
    CUDA_OK(cudaMemcpyAsync(d_tabs, tabs.data(), tabs.size() * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    return EDEN_OK;
}

int encode_common(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                  const double* bits, const double* delta, const uint64_t* seeds,
                  uint8_t* const* codes, float* scales)
{
    if (!ctx || !x || !seeds || !codes || !scales || ld_x < d) return EDEN_ERR_INVALID_ARG;
    std::vector<ClientPlan> plan;
    int rc = plan_clients(d, n, bits, delta, plan);
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        if (!codes[c] || ((uintptr_t)codes[c] & 15u)) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    CallLayout lay;
    rc = carve(ctx, d, n, delta != nullptr, lay);
    if (rc) return rc;
    std::vector<Group> groups;
    SelectionAhead ahead(ctx);
    ahead.plan_arena(plan, d, lay);
    rc = make_groups(ctx, plan, d, lay.work_bytes, groups, ahead.on);
    if (rc == EDEN_ERR_WORKSPACE && ahead.on) {
        ahead.cancel(lay);
        groups.clear();
        rc = make_groups(ctx, plan, d, lay.work_bytes, groups);
    }
    if (rc) return rc;
    const FixedLayout f = fixed_layout(d);
    const bool x_aligned = ((uintptr_t)x & 15u) == 0 && (ld_x & 3u) == 0;

    // descriptors in processing order
    std::vector<ClientDesc> descs;
    descs.reserve(n);
    ctx->order.clear();
    std::vector<uint32_t> group_start;
    for (const Group& g : groups) {
        group_start.push_back((uint32_t)descs.size());
        uint64_t off = 0;
        for (uint32_t m : g.members) {
            const ClientPlan& p = plan[m];
            ClientDesc cd;
            std::memset(&cd, 0, sizeof(cd));
            cd.work = p.needs_work ? (float*)(ctx->ws + lay.work_off + off) : nullptr;
            if (p.needs_work) off += work_buffer_bytes(p.D);
            cd.src = p.subbit ? cd.work : x + (uint64_t)p.index * ld_x;
            cd.codes = (uint32_t*)codes[p.index];
            cd.recv = nullptr;
            cd.recv_shift = 10;
            cd.seed = seeds[p.index];
            cd.valid = p.k;
            cd.d = d;
            cd.W = (uint32_t)p.W;
            cd.L = (uint32_t)p.L;
            cd.subbit = p.subbit;
            cd.index = p.index;
            cd.coin_thr = p.coin_thr;
            cd.extra_scale = p.subbit ? (double)d / (double)p.k : 1.0;
            cd.mean_scale = 1.0;
            descs.push_back(cd);
            ctx->order.push_back(p.index);
        }
    }
    ClientDesc* d_descs = (ClientDesc*)(ctx->ws + lay.descs_off);
    ClientState* d_states = (ClientState*)(ctx->ws + lay.states_off);
    uint32_t* d_status = (uint32_t*)(ctx->ws + f.status);
    ctx->states_off = lay.states_off;
    if (delta) {
        rc = upload_uniform_tables(ctx, lay, plan, ctx->order, descs);
        if (rc) return rc;
    }
    rc = upload_descs_and_clear_states(ctx, lay, descs);
    if (rc) return rc;

    // Small rounds (the paper's federated-learning sizes) are a handful of launches of a few
    // microseconds each: there the row pass writes the scales itself and k_enc_scale is not
    // launched.  Needs every group on the register-blocked path.
    bool fold = !ctx->row_staging;
    uint64_t fold_tiles = 0;
    for (const Group& g : groups) {
        fold = fold && fast_eligible(ctx, g) && (x_aligned || g.subbit);
        fold_tiles += (uint64_t)g.members.size() << (g.L > kFastTileLog ? g.L - kFastTileLog : 0);
    }
    fold = fold && fold_tiles <= kFoldMaxTiles;
    // selection jobs of a b < 1 group; *work_end gets the bytes its work buffers take
    auto selection_jobs = [&](size_t gi, std::vector<SelJob>& jobs, uint64_t* work_end, uint64_t* kept) {
        const Group& g = groups[gi];
        const uint32_t first = group_start[gi], gn = (uint32_t)g.members.size();
        jobs.resize(gn);
        *work_end = 0;
        *kept = 0;
        for (uint32_t j = 0; j < gn; ++j) {
            const ClientPlan& p = plan[g.members[j]];
            std::memset(&jobs[j], 0, sizeof(SelJob));
            jobs[j].seed = seeds[p.index];
            jobs[j].d = d;
            jobs[j].k = p.k;
            jobs[j].in = x + (uint64_t)p.index * ld_x;
            jobs[j].out = descs[first + j].work;
            *work_end += work_buffer_bytes(p.D);
            *kept += p.k;
        }
    };
    if (ahead.on) {
        rc = ahead.begin(groups.size());
        uint64_t off = ahead.arena_off;
        for (size_t gi = 0; gi < groups.size() && rc == EDEN_OK; ++gi) {
            if (!groups[gi].subbit) continue;
            std::vector<SelJob> jobs;
            uint64_t work_end, kept;
            selection_jobs(gi, jobs, &work_end, &kept);
            rc = start_selection_batch(ctx, ctx->ws + off, d, jobs, ahead.batches[gi]);
            if (rc == EDEN_OK) rc = ahead.mark(gi);
            off += groups[gi].members.size() * sel_scratch_bytes(ctx, d);
        }
        ahead.end();
        if (rc) return rc;
    }
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        const uint32_t first = group_start[gi], gn = (uint32_t)g.members.size();
        if (g.subbit) {
            // exact-size masks of all members, then gather their kept coordinates
            std::vector<SelJob> jobs;
            uint64_t work_end, kept;
            selection_jobs(gi, jobs, &work_end, &kept);
            SelBatch batch;
            if (ahead.on) {
                rc = ahead.wait(gi);
                batch = ahead.batches[gi];
            } else {
                rc = start_selection_batch(ctx, ctx->ws + lay.work_off + work_end, d, jobs, batch);
            }
            if (rc) return rc;
            if (batch.two_pass)
                LAUNCH(ctx, "sel_compact", 4.0 * gn * (double)d + 4.0 * (double)kept, k_selc_compact,
                       dim3((batch.grid + kSelThreads / 32 - 1) / (kSelThreads / 32), gn), kSelThreads, 0,
                       (const SelJob*)batch.d_jobs, (uint64_t)batch.grid);
            else
                LAUNCH(ctx, "sel_compact", 4.0 * gn * (double)d + 4.0 * (double)kept, k_selb_compact,
                       dim3(batch.grid, gn), kSelThreads, 0, (const SelJob*)batch.d_jobs);
        }
        if (fast_eligible(ctx, g) && (x_aligned || g.subbit)) {
            rc = fast_encode_group(ctx, plan, g, descs.data() + first, d_descs + first, d_states + first, d, d_status,
                                   fold ? scales : nullptr);
            if (rc) return rc;
        } else if (g.L <= kGenericTileLog) {
            const PassGeom rg = row_geom(g.L);
            LAUNCH(ctx, "enc_single", gn * (4.0 * std::min<uint64_t>(d, 1ull << g.L) + (double)(1ull << g.L) / 8), k_enc_last<true>, dim3(1, gn), kGenericThreads, sizeof(float) << g.L,
                   d_descs + first, d_states + first, rg);
        } else {
            const int lc = kGenericTileLog;
            std::vector<BitRange> cols;
            column_ranges(g.L, lc, 8, cols);
            for (size_t pi = 0; pi < cols.size(); ++pi) {
                const PassGeom cg = column_geom(cols[pi]);
                const unsigned tiles = (unsigned)((1ull << g.L) >> cg.lt);
                if (pi == 0)
                    LAUNCH(ctx, "enc_first", gn * (4.0 * std::min<uint64_t>(d, 1ull << g.L) + 4.0 * (double)(1ull << g.L)), k_enc_first, dim3(tiles, gn), kGenericThreads, sizeof(float) << cg.lt,
                           d_descs + first, d_states + first, cg);
                else
                    LAUNCH(ctx, "mid", gn * 8.0 * (double)(1ull << g.L), k_mid, dim3(tiles, gn), kGenericThreads, sizeof(float) << cg.lt,
                           d_descs + first, cg);
            }
            const PassGeom rg = row_geom(lc);
            LAUNCH(ctx, "enc_last", gn * (4.0 + code_bits_per_coord(plan, g) / 8.0) * (double)(1ull << g.L), k_enc_last<false>, dim3((unsigned)((1ull << g.L) >> lc), gn), kGenericThreads,
                   sizeof(float) << lc, d_descs + first, d_states + first, rg);
        }
    }
    if (!fold)
        LAUNCH(ctx, "enc_scale", n * 20.0, k_enc_scale, (n + 127) / 128, 128, 0, d_descs, d_states, scales, n, d_status);
    return EDEN_OK;
}

}  // namespace

extern "C" int eden_encode(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                           const double* bits, const uint64_t* seeds,
                           uint8_t* const* codes, float* scales)
{
    if (!bits) return EDEN_ERR_INVALID_ARG;
    return encode_common(ctx, x, ld_x, d, n, bits, nullptr, seeds, codes, scales);
}

extern "C" int eden_encode_uniform(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                                   const double* delta, const uint64_t* seeds,
                                   int8_t* const* index, float* scales)
{
    if (!delta) return EDEN_ERR_INVALID_ARG;
    return encode_common(ctx, x, ld_x, d, n, nullptr, delta, seeds, (uint8_t* const*)index, scales);
}

// ------------------------------------------------------------------------------------
// receiver
// ------------------------------------------------------------------------------------
// recv_shift: log2 of the coordinates one bit of a recv_masks bitmap stands for: 10 for
// packets (Section 4.2); 0 for a bitmap with one bit per rotated coordinate (one-bit codes only).
static int decode_common(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                         const double* bits, const double* delta, const uint64_t* seeds,
                         const uint32_t* const* recv_masks, uint64_t d, uint32_t n,
                         float* out, uint64_t divisor /* 0: accumulate into out; else overwrite out with the sum / divisor */,
                         uint32_t recv_shift = 10, const uint32_t* recv_ones = nullptr /* per client: set bits of its bitmap, if known */)
{
    if (!ctx || !codes || !scales || !seeds || !out || ((uintptr_t)out & 3u)) return EDEN_ERR_INVALID_ARG;
    const bool mean = divisor != 0;
    std::vector<ClientPlan> plan;
    int rc = plan_clients(d, n, bits, delta, plan);
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        if (!codes[c] || ((uintptr_t)codes[c] & 3u)) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    CallLayout lay;
    rc = carve(ctx, d, n, delta != nullptr, lay);
    if (rc) return rc;
    std::vector<Group> groups;
    SelectionAhead ahead(ctx);
    ahead.plan_arena(plan, d, lay);
    rc = make_groups(ctx, plan, d, lay.work_bytes, groups, ahead.on);
    if (rc == EDEN_ERR_WORKSPACE && ahead.on) {
        ahead.cancel(lay);
        groups.clear();
        rc = make_groups(ctx, plan, d, lay.work_bytes, groups);
    }
    if (rc) return rc;
    const FixedLayout f = fixed_layout(d);
    // the register-blocked last pass moves `out` 16 bytes at a time; a vector that is not
    // 16-byte aligned goes through the shape-generic kernels, whose accesses are scalar
    const bool out_aligned = ((uintptr_t)out & 15u) == 0;

    std::vector<ClientDesc> descs;
    descs.reserve(n);
    ctx->order.clear();
    std::vector<uint32_t> group_start;
    std::vector<uint64_t> group_work_end;       // bytes of the work region the group's buffers take
    for (const Group& g : groups) {
        group_start.push_back((uint32_t)descs.size());
        group_work_end.push_back(0);
        uint64_t off = 0;
        for (uint32_t m : g.members) {
            const ClientPlan& p = plan[m];
            ClientDesc cd;
            std::memset(&cd, 0, sizeof(cd));
            cd.work = p.needs_work ? (float*)(ctx->ws + lay.work_off + off) : nullptr;
            if (p.needs_work) off += work_buffer_bytes(p.D);
            group_work_end.back() = off;
            cd.src = nullptr;
            cd.codes = (uint32_t*)codes[p.index];
            cd.recv = recv_masks ? recv_masks[p.index] : nullptr;
            cd.recv_shift = recv_shift;
            cd.recv_ones = recv_ones ? recv_ones[p.index] : 0u;
            cd.seed = seeds[p.index];
            cd.valid = p.k;
            cd.d = d;
            cd.W = (uint32_t)p.W;
            cd.L = (uint32_t)p.L;
            cd.subbit = p.subbit;
            cd.index = p.index;
            cd.coin_thr = p.coin_thr;
            cd.extra_scale = 1.0;
            cd.mean_scale = mean ? 1.0 / (double)divisor : 1.0;
            descs.push_back(cd);
            ctx->order.push_back(p.index);
        }
    }
    ClientDesc* d_descs = (ClientDesc*)(ctx->ws + lay.descs_off);
    ClientState* d_states = (ClientState*)(ctx->ws + lay.states_off);
    uint32_t* d_status = (uint32_t*)(ctx->ws + f.status);
    ctx->states_off = lay.states_off;
    if (delta) {
        rc = upload_uniform_tables(ctx, lay, plan, ctx->order, descs);
        if (rc) return rc;
    }
    rc = upload_descs_and_clear_states(ctx, lay, descs);
    if (rc) return rc;
    // small rounds: the receiver's row pass computes p and the factor itself (see encode_common)
    bool fold = true;
    uint64_t fold_tiles = 0;
    for (const Group& g : groups) {
        fold = fold && fast_eligible(ctx, g) && (out_aligned || g.subbit) &&
               ((1ull << g.L) >> recv_shift) <= 32ull * kFoldMaxMaskWords;
        fold_tiles += (uint64_t)g.members.size() << (g.L > kFastTileLog ? g.L - kFastTileLog : 0);
    }
    fold = fold && fold_tiles <= kFoldMaxTiles;
    if (!fold)
        LAUNCH(ctx, "dec_prep", n * 8.0, k_dec_prep, n, 256, 0, d_descs, d_states, scales, d_status);

    // the first group with b >= 1 covers every output coordinate, so for the mean it may
    // overwrite; everything after it accumulates
    bool written = !mean;
    if (mean && (groups.empty() || groups[0].subbit)) {
        CUDA_OK(cudaMemsetAsync(out, 0, d * sizeof(float), ctx->stream));
        written = true;
    }
    // selection jobs of a b < 1 group; *work_end gets the bytes its work buffers take
    auto selection_jobs = [&](size_t gi, std::vector<SelJob>& jobs, uint64_t* work_end, uint64_t* kept) {
        const Group& g = groups[gi];
        const uint32_t first = group_start[gi], gn = (uint32_t)g.members.size();
        jobs.resize(gn);
        *work_end = 0;
        *kept = 0;
        for (uint32_t j = 0; j < gn; ++j) {
            const ClientPlan& p = plan[g.members[j]];
            std::memset(&jobs[j], 0, sizeof(SelJob));
            jobs[j].seed = seeds[p.index];
            jobs[j].d = d;
            jobs[j].k = p.k;
            jobs[j].in = descs[first + j].work;
            *work_end += work_buffer_bytes(p.D);
            *kept += p.k;
        }
    };
    if (ahead.on) {
        rc = ahead.begin(groups.size());
        uint64_t off = ahead.arena_off;
        for (size_t gi = 0; gi < groups.size() && rc == EDEN_OK; ++gi) {
            if (!groups[gi].subbit) continue;
            std::vector<SelJob> jobs;
            uint64_t work_end, kept;
            selection_jobs(gi, jobs, &work_end, &kept);
            rc = start_selection_batch(ctx, ctx->ws + off, d, jobs, ahead.batches[gi]);
            if (rc == EDEN_OK) rc = ahead.mark(gi);
            off += groups[gi].members.size() * sel_scratch_bytes(ctx, d);
        }
        ahead.end();
        if (rc) return rc;
    }
    for (size_t gi = 0; gi < groups.size(); ++gi) {
        const Group& g = groups[gi];
        const uint32_t first = group_start[gi], gn = (uint32_t)g.members.size();
        int mode = g.subbit ? OUT_YHAT : (written ? OUT_ACC : OUT_WRITE);
        SelBatch batch{nullptr, 0, 0, false, {}};
        uint64_t kept = 0;
        if (g.subbit) {
            // exact-size masks of all members (the estimates of their kept coordinates will
            // be written to their work buffers and scattered from there)
            std::vector<SelJob> jobs;
            uint64_t work_end;
            selection_jobs(gi, jobs, &work_end, &kept);
            if (ahead.on) {
                rc = ahead.wait(gi);
                batch = ahead.batches[gi];
            } else {
                rc = start_selection_batch(ctx, ctx->ws + lay.work_off + work_end, d, jobs, batch);
            }
            if (rc) return rc;
        }
        // with OUT_YHAT every member writes its own estimate: one block row per member
        const uint32_t loop_n = g.subbit ? 1u : gn;
        const unsigned rows = g.subbit ? gn : 1u;
        if (fast_eligible(ctx, g) && (out_aligned || g.subbit)) {
            rc = fast_decode_group(ctx, plan, g, d_descs + first, d_states + first, out, d, mode,
                                   (float*)(ctx->ws + lay.work_off + group_work_end[gi]),
                                   lay.work_bytes - group_work_end[gi], fold ? scales : nullptr, d_status);
            if (rc) return rc;
        } else if (g.L <= kGenericTileLog) {
            const PassGeom rg = row_geom(g.L);
            // many small clients: spread them over block rows with partial sums (see
            // fast_decode_group), up to about two blocks per SM
            const uint64_t stride = align_up(d, 64);
            float* part = (float*)(ctx->ws + lay.work_off + group_work_end[gi]);
            const uint64_t part_bytes = lay.work_bytes - group_work_end[gi];
            uint32_t split_rows = 1, per = gn;
            if (!g.subbit && gn >= 4) {
                const uint32_t want = std::min<uint32_t>(gn / 2, 2u * (unsigned)ctx->sm_count);
                per = (gn + want - 1) / want;
                split_rows = (gn + per - 1) / per;
                if (split_rows < 2 || (uint64_t)split_rows * stride * sizeof(float) > part_bytes) { split_rows = 1; per = gn; }
            }
            if (split_rows > 1) {
                LAUNCH(ctx, "dec_single", gn * code_bits_per_coord(plan, g) / 8.0 * (double)(1ull << g.L) + split_rows * 4.0 * d,
                       k_dec_last<true>, dim3(1, split_rows), kGenericThreads, sizeof(float) << g.L,
                       d_descs + first, d_states + first, per, rg, part, d, (int)OUT_PART, gn, stride);
                LAUNCH(ctx, "dec_sum", (split_rows + (mode == OUT_ACC ? 2.0 : 1.0)) * 4.0 * (double)d, k_sum_partials,
                       (unsigned)((d + 1023) / 1024), 256, 0, (const float*)part, split_rows, stride, d, out,
                       mode == OUT_ACC ? 1 : 0);
            } else {
                LAUNCH(ctx, "dec_single", gn * code_bits_per_coord(plan, g) / 8.0 * (double)(1ull << g.L) + 4.0 * d, k_dec_last<true>, dim3(1, rows), kGenericThreads, sizeof(float) << g.L,
                       d_descs + first, d_states + first, loop_n, rg, out, d, mode, gn, (uint64_t)0);
            }
        } else {
            const int lc = kGenericTileLog;
            LAUNCH(ctx, "dec_first", gn * (4.0 + code_bits_per_coord(plan, g) / 8.0) * (double)(1ull << g.L), k_dec_first, dim3((unsigned)((1ull << g.L) >> lc), gn), kGenericThreads,
                   sizeof(float) << lc, d_descs + first, row_geom(lc));
            std::vector<BitRange> cols;
            column_ranges(g.L, lc, 8, cols);
            for (size_t pi = 0; pi < cols.size(); ++pi) {
                const PassGeom cg = column_geom(cols[pi]);
                const unsigned tiles = (unsigned)((1ull << g.L) >> cg.lt);
                if (pi + 1 < cols.size())
                    LAUNCH(ctx, "mid", gn * 8.0 * (double)(1ull << g.L), k_mid, dim3(tiles, gn), kGenericThreads, sizeof(float) << cg.lt,
                           d_descs + first, cg);
                else
                    LAUNCH(ctx, "dec_last", gn * 4.0 * (double)(1ull << g.L) + (mode == OUT_ACC ? 8.0 : 4.0) * std::min<uint64_t>(d, 1ull << g.L), k_dec_last<false>, dim3(tiles, rows), kGenericThreads, sizeof(float) << cg.lt,
                           d_descs + first, d_states + first, loop_n, cg, out, d, mode, gn, (uint64_t)0);
            }
        }
        if (g.subbit) {
            if (batch.two_pass)
                LAUNCH(ctx, "sel_scatter", 8.0 * (double)kept + 4.0 * (double)kept, k_selc_scatter,
                       (batch.grid + kSelThreads / 32 - 1) / (kSelThreads / 32), kSelThreads, 0,
                       (const SelJob*)batch.d_jobs, gn, d, out, (uint64_t)batch.grid);
            else
                LAUNCH(ctx, "sel_scatter", 8.0 * (double)kept + 4.0 * (double)kept, k_selb_scatter, batch.grid,
                       kSelThreads, 0, (const SelJob*)batch.d_jobs, gn, d, out);
        } else {
            written = true;
        }
    }
    return EDEN_OK;
}

extern "C" int eden_decode_accumulate(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                                      const double* bits, const uint64_t* seeds,
                                      const uint32_t* const* recv_masks,
                                      uint64_t d, uint32_t n, float* acc, uint32_t* n_used)
{
    if (!bits) return EDEN_ERR_INVALID_ARG;
    const int rc = decode_common(ctx, codes, scales, bits, nullptr, seeds, recv_masks, d, n, acc, 0);
    if (rc == EDEN_OK && n_used) *n_used += n;
    return rc;
}

extern "C" int eden_decode_accumulate_uniform(eden_ctx* ctx, const int8_t* const* index, const float* scales,
                                              const double* delta, const uint64_t* seeds,
                                              const uint32_t* const* recv_masks,
                                              uint64_t d, uint32_t n, float* acc, uint32_t* n_used)
{
    if (!delta) return EDEN_ERR_INVALID_ARG;
    const int rc = decode_common(ctx, (const uint8_t* const*)index, scales, nullptr, delta, seeds, recv_masks,
                                 d, n, acc, 0);
    if (rc == EDEN_OK && n_used) *n_used += n;
    return rc;
}

extern "C" int eden_mean_uniform(eden_ctx* ctx, const int8_t* const* index, const float* scales,
                                 const double* delta, const uint64_t* seeds,
                                 const uint32_t* const* recv_masks,
                                 uint64_t d, uint32_t n, float* mean)
{
    if (!delta) return EDEN_ERR_INVALID_ARG;
    return decode_common(ctx, (const uint8_t* const*)index, scales, nullptr, delta, seeds, recv_masks, d, n,
                         mean, n);
}

// How often each index value occurs in each client's message (Section 4.3: what an entropy
// coder's model, and the estimate of the coded length, are built from).
extern "C" int eden_index_histogram(eden_ctx* ctx, const int8_t* const* index, uint64_t d, uint32_t n,
                                    uint32_t* hist)
{
    if (!ctx || !index || !hist || d == 0 || n == 0) return EDEN_ERR_INVALID_ARG;
    if (d > EDEN_MAX_DIM) return EDEN_ERR_TOO_LARGE;
    for (uint32_t c = 0; c < n; ++c)
        if (!index[c] || ((uintptr_t)index[c] & 15u)) return EDEN_ERR_INVALID_ARG;
    CUDA_OK(cudaSetDevice(ctx->device));
    const uint64_t D = eden_rot_dim(d, 1.0);
    const uint64_t ptr_bytes = align_up(sizeof(const int8_t*) * (uint64_t)n, 256);
    const FixedLayout f = fixed_layout(d);
    if (f.end + ptr_bytes > ctx->ws_bytes) return EDEN_ERR_WORKSPACE;
    const int8_t** d_ptrs = (const int8_t**)(ctx->ws + f.end);
    CUDA_OK(cudaMemcpyAsync(d_ptrs, index, sizeof(const int8_t*) * (uint64_t)n, cudaMemcpyHostToDevice, ctx->stream));
    CUDA_OK(cudaMemsetAsync(hist, 0, 256ull * sizeof(uint32_t) * n, ctx->stream));
    const uint64_t per_block = (uint64_t)kHistThreads * kHistBytesPerThread;
    const unsigned blocks = (unsigned)std::min<uint64_t>((D + per_block - 1) / per_block, 4ull * ctx->sm_count);
    LAUNCH(ctx, "index_hist", (double)n * (double)D, k_index_hist, dim3(blocks, n), kHistThreads, 0,
           (const int8_t* const*)d_ptrs, D, hist);
    return EDEN_OK;
}

extern "C" int eden_mean(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                         const double* bits, const uint64_t* seeds,
                         const uint32_t* const* recv_masks,
                         uint64_t d, uint32_t n, float* mean)
{
    if (!bits) return EDEN_ERR_INVALID_ARG;
    return decode_common(ctx, codes, scales, bits, nullptr, seeds, recv_masks, d, n, mean, n);
}

extern "C" int eden_mean_partial(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                                 const double* bits, const uint64_t* seeds,
                                 const uint32_t* const* recv_masks,
                                 uint64_t d, uint32_t n, uint64_t n_total, float* partial)
{
    if (!bits || n_total < n) return EDEN_ERR_INVALID_ARG;
    return decode_common(ctx, codes, scales, bits, nullptr, seeds, recv_masks, d, n, partial, n_total);
}

extern "C" int eden_sparsification_mask(eden_ctx* ctx, uint64_t seed, uint64_t d, double bits,
                                        uint32_t* mask_bits)
{
    if (!ctx || !mask_bits || d == 0 || !(bits > 0.0) || !(bits < 1.0)) return EDEN_ERR_INVALID_ARG;
    if (d > EDEN_MAX_DIM) return EDEN_ERR_TOO_LARGE;
    CUDA_OK(cudaSetDevice(ctx->device));
    const FixedLayout f = fixed_layout(d);
    if (f.end > ctx->ws_bytes) return EDEN_ERR_WORKSPACE;
    // where the workspace has room for it, the batched selection with one job (one pass over
    // the keys, see start_selection_batch), whose mask bitmap is the answer
    const uint64_t region = align_up(f.end, 256);
    if (two_pass_selection(ctx, d) && region + sel_scratch_bytes(ctx, d) <= ctx->ws_bytes) {
        std::vector<SelJob> jobs(1);
        std::memset(&jobs[0], 0, sizeof(SelJob));
        jobs[0].seed = seed;
        jobs[0].d = d;
        jobs[0].k = eden_kept_count(d, bits);
        SelBatch batch;
        const int rc = start_selection_batch(ctx, ctx->ws + region, d, jobs, batch);
        if (rc) return rc;
        CUDA_OK(cudaMemcpyAsync(mask_bits, batch.keep[0], (d + 31) / 32 * sizeof(uint32_t), cudaMemcpyDeviceToDevice,
                                ctx->stream));
        return EDEN_OK;
    }
    const int rc = run_selection(ctx, f, seed, d, eden_kept_count(d, bits));
    if (rc) return rc;
    const unsigned grid = (unsigned)(((d + 3) / 4 + kSelThreads - 1) / kSelThreads);
    LAUNCH(ctx, "sel_mask_bits", d / 8.0, k_sel_apply<SEL_MASK_BITS>, grid, kSelThreads, 0, seed, d,
           (const MaskSelect*)(ctx->ws + f.sel), (const unsigned long long*)(ctx->ws + f.chunks),
           (const float*)nullptr, (float*)nullptr, mask_bits);
    return EDEN_OK;
}

// ------------------------------------------------------------------------------------
// Section 4.1, the other order: sparsification after the rotation.  The sender runs the
// one-bit encode of the whole vector and keeps the codes of a random mask over the
// rotated coordinates; the receiver spreads them back, takes the mask as the pattern of
// what arrived (Lemma 4.3) and decodes as under loss.  The full code streams, the masks
// and the selection scratch live at the tail of the workspace for the call.
// ------------------------------------------------------------------------------------
extern "C" uint64_t eden_after_kept_count(uint64_t d, double bits)
{
    return eden_kept_count(eden_rot_dim(d, 1.0), bits);
}

extern "C" uint64_t eden_after_code_bytes(uint64_t d, double bits)
{
    const uint64_t words = (eden_after_kept_count(d, bits) + 31) / 32;
    return (words * 4 + 15) / 16 * 16;
}

namespace {

uint64_t after_tail_bytes(const eden_ctx* ctx, uint64_t D, uint32_t n)
{
    return (uint64_t)n * (align_up(eden_code_bytes(D, 1.0), 256) + sel_scratch_bytes(ctx, D) + 256) + 4096;
}

struct AfterCall {
    std::vector<uint8_t*> full;          // full one-bit code stream of each client (device)
    SelBatch batch;
    uint64_t D, head_bytes;              // head_bytes: what is left of the workspace for the ordinary call
    unsigned chunk_grid;
};

// carves the tail of the workspace and starts the mask selection over the D rotated coordinates
int after_begin(eden_ctx* ctx, uint64_t d, uint32_t n, const double* bits, const uint64_t* seeds, AfterCall& ac)
{
    if (!ctx || !bits || !seeds || d == 0 || n == 0) return EDEN_ERR_INVALID_ARG;
    if (d > EDEN_MAX_DIM) return EDEN_ERR_TOO_LARGE;
    for (uint32_t c = 0; c < n; ++c)
        if (!(bits[c] > 0.0) || !(bits[c] < 1.0)) return EDEN_ERR_UNSUPPORTED_BITS;
    ac.D = eden_rot_dim(d, 1.0);
    if (!two_pass_selection(ctx, ac.D)) return EDEN_ERR_TOO_LARGE;      // the bitmap form of the selection only
    CUDA_OK(cudaSetDevice(ctx->device));
    const uint64_t tail = after_tail_bytes(ctx, ac.D, n);
    if (tail + fixed_layout(1).end > ctx->ws_bytes) return EDEN_ERR_WORKSPACE;
    ac.head_bytes = (ctx->ws_bytes - tail) / 256 * 256;
    char* p = ctx->ws + ac.head_bytes;
    const uint64_t full_bytes = align_up(eden_code_bytes(ac.D, 1.0), 256);
    ac.full.resize(n);
    for (uint32_t c = 0; c < n; ++c) ac.full[c] = (uint8_t*)(p + full_bytes * c);
    ac.chunk_grid = (unsigned)(((ac.D + kSelChunk - 1) / kSelChunk + kSelThreads / 32 - 1) / (kSelThreads / 32));
    return EDEN_OK;
}

// starts the selection with the jobs' stream pointers set (in -> out as k_after_rotation_bits reads them)
int after_select(eden_ctx* ctx, AfterCall& ac, uint32_t n, const double* bits, const uint64_t* seeds,
                 const std::vector<const void*>& in, const std::vector<void*>& out)
{
    std::vector<SelJob> jobs(n);
    for (uint32_t c = 0; c < n; ++c) {
        std::memset(&jobs[c], 0, sizeof(SelJob));
        jobs[c].seed = seeds[c];
        jobs[c].d = ac.D;
        jobs[c].k = eden_kept_count(ac.D, bits[c]);
        jobs[c].in = (const float*)in[c];
        jobs[c].out = (float*)out[c];
    }
    char* region = ctx->ws + ac.head_bytes + align_up(eden_code_bytes(ac.D, 1.0), 256) * (uint64_t)n;
    return start_selection_batch(ctx, region, ac.D, jobs, ac.batch);
}

}  // namespace

extern "C" uint64_t eden_after_workspace_bytes(uint64_t d, uint32_t n)
{
    const uint64_t D = eden_rot_dim(d ? d : 1, 1.0);
    const uint64_t n_chunks = (D + kSelChunk - 1) / kSelChunk;
    // the larger of the two selection forms, as eden_workspace_bytes reserves it
    const uint64_t sel = 256 + kBatchHistBytes + align_up(n_chunks * sizeof(unsigned long long), 256) +
                         align_up(sizeof(SelJob), 256) + kCandBytes + keep_bitmap_bytes(D);
    return eden_workspace_bytes(d, n) +
           (uint64_t)(n ? n : 1) * (align_up(eden_code_bytes(D, 1.0), 256) + sel + 256) + 4096 + 512;
}

extern "C" int eden_encode_sparsify_after(eden_ctx* ctx, const float* x, uint64_t ld_x, uint64_t d, uint32_t n,
                                          const double* bits, const uint64_t* seeds,
                                          uint8_t* const* codes, float* scales)
{
    if (!codes) return EDEN_ERR_INVALID_ARG;
    AfterCall ac;
    int rc = after_begin(ctx, d, n, bits, seeds, ac);
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        if (!codes[c] || ((uintptr_t)codes[c] & 15u)) return EDEN_ERR_INVALID_ARG;
    std::vector<const void*> in(n);
    std::vector<void*> out(n);
    for (uint32_t c = 0; c < n; ++c) {
        in[c] = ac.full[c];
        out[c] = codes[c];
    }
    // the whole vector with one bit per rotated coordinate, exactly as for b = 1
    const std::vector<double> one(n, 1.0);
    const uint64_t saved = ctx->ws_bytes;
    ctx->ws_bytes = ac.head_bytes;
    rc = encode_common(ctx, x, ld_x, d, n, one.data(), nullptr, seeds, ac.full.data(), scales);
    ctx->ws_bytes = saved;
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        CUDA_OK(cudaMemsetAsync(codes[c], 0, eden_after_code_bytes(d, bits[c]), ctx->stream));
    rc = after_select(ctx, ac, n, bits, seeds, in, out);
    if (rc) return rc;
    const uint64_t n_chunks = (ac.D + kSelChunk - 1) / kSelChunk;
    LAUNCH(ctx, "after_pack", n * (double)ac.D / 4.0, k_after_rotation_bits<true>, dim3(ac.chunk_grid, n), kSelThreads, 0,
           (const SelJob*)ac.batch.d_jobs, n_chunks);
    return EDEN_OK;
}

static int after_decode(eden_ctx* ctx, const uint8_t* const* codes, const float* scales, const double* bits,
                        const uint64_t* seeds, uint64_t d, uint32_t n, float* out, uint64_t divisor)
{
    if (!codes || !scales || !out) return EDEN_ERR_INVALID_ARG;
    AfterCall ac;
    int rc = after_begin(ctx, d, n, bits, seeds, ac);
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        if (!codes[c] || ((uintptr_t)codes[c] & 3u)) return EDEN_ERR_INVALID_ARG;
    std::vector<const void*> in(n);
    std::vector<void*> full(n);
    for (uint32_t c = 0; c < n; ++c) {
        in[c] = codes[c];
        full[c] = ac.full[c];
    }
    rc = after_select(ctx, ac, n, bits, seeds, in, full);
    if (rc) return rc;
    const uint64_t n_chunks = (ac.D + kSelChunk - 1) / kSelChunk;
    LAUNCH(ctx, "after_unpack", n * (double)ac.D / 4.0, k_after_rotation_bits<false>, dim3(ac.chunk_grid, n), kSelThreads, 0,
           (const SelJob*)ac.batch.d_jobs, n_chunks);
    // the mask is the pattern of what arrived: the receiver counts it and divides by p (Lemma 4.3)
    const std::vector<double> one(n, 1.0);
    const uint64_t saved = ctx->ws_bytes;
    ctx->ws_bytes = ac.head_bytes;
    std::vector<uint32_t> kept(n);                     // the masks have exactly this many ones (Section 4.1)
    for (uint32_t c = 0; c < n; ++c) kept[c] = (uint32_t)eden_kept_count(ac.D, bits[c]);
    rc = decode_common(ctx, (const uint8_t* const*)ac.full.data(), scales, one.data(), nullptr, seeds,
                       ac.batch.keep.data(), d, n, out, divisor, 0, kept.data());
    ctx->ws_bytes = saved;
    return rc;
}

extern "C" int eden_mean_sparsify_after(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                                        const double* bits, const uint64_t* seeds,
                                        uint64_t d, uint32_t n, float* mean)
{
    return after_decode(ctx, codes, scales, bits, seeds, d, n, mean, n);
}

extern "C" int eden_decode_accumulate_sparsify_after(eden_ctx* ctx, const uint8_t* const* codes, const float* scales,
                                                     const double* bits, const uint64_t* seeds,
                                                     uint64_t d, uint32_t n, float* acc, uint32_t* n_used)
{
    const int rc = after_decode(ctx, codes, scales, bits, seeds, d, n, acc, 0);
    if (rc == EDEN_OK && n_used) *n_used += n;
    return rc;
}

// ------------------------------------------------------------------------------------
// host-buffer variants: stage through the tail of the workspace
// ------------------------------------------------------------------------------------
extern "C" uint64_t eden_host_workspace_bytes(uint64_t d, uint32_t n)
{
    const uint64_t D = 1ull << ceil_log2(d ? d : 1);
    // vectors, codes at 8 bits, scales, masks, mean
    const uint64_t staging = (uint64_t)n * align_up(d * sizeof(float), 256) +
                             (uint64_t)n * align_up(D, 256) + align_up(n * sizeof(float), 256) +
                             (uint64_t)n * align_up(((D + 1023) / 1024 + 31) / 32 * 4, 256) +
                             align_up(d * sizeof(float), 256) + 4096;
    return eden_workspace_bytes(d, n) + staging;
}

namespace {
struct Staging {
    char* base;
    uint64_t left;
    void* take(uint64_t bytes)
    {
        bytes = align_up(bytes, 256);
        if (bytes > left) return nullptr;
        left -= bytes;
        return base + left;   // carve downwards from the end of the workspace
    }
};
}  // namespace

extern "C" int eden_encode_host(eden_ctx* ctx, const float* x_host, uint64_t ld_x, uint64_t d, uint32_t n,
                                const double* bits, const uint64_t* seeds,
                                uint8_t* const* codes_host, float* scales_host)
{
    if (!ctx || !x_host || !bits || !seeds || !codes_host || !scales_host || ld_x < d || d == 0 || n == 0)
        return EDEN_ERR_INVALID_ARG;
    for (uint32_t c = 0; c < n; ++c)
        if (eden_code_width(bits[c]) == 0) return EDEN_ERR_UNSUPPORTED_BITS;
    CUDA_OK(cudaSetDevice(ctx->device));
    Staging st{ctx->ws, ctx->ws_bytes};
    const uint64_t row = align_up(d * sizeof(float), 256) / sizeof(float);
    float* x_dev = (float*)st.take((uint64_t)n * row * sizeof(float));
    float* scales_dev = (float*)st.take(n * sizeof(float));
    if (!x_dev || !scales_dev) return EDEN_ERR_WORKSPACE;
    std::vector<uint8_t*> codes_dev(n);
    for (uint32_t c = 0; c < n; ++c) {
        codes_dev[c] = (uint8_t*)st.take(eden_code_bytes(d, bits[c]));
        if (!codes_dev[c]) return EDEN_ERR_WORKSPACE;
    }
    const uint64_t saved = ctx->ws_bytes;
    // Large inputs go through in chunks of clients: the upload of the next chunk, the
    // kernels of this one and the download of the previous chunk's codes overlap.
    const uint64_t row_bytes = d * sizeof(float);
    const uint32_t chunk = (uint32_t)std::max<uint64_t>(1, (32ull << 20) / row_bytes);
    if (n > chunk && (uint64_t)n * row_bytes >= (64ull << 20)) {
        if (!ctx->copy_in) {
            CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking));
            CUDA_OK(cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking));
        }
        const uint32_t n_chunks = (n + chunk - 1) / chunk;
        while (ctx->sync_events.size() < 2ull * n_chunks + 2) {
            cudaEvent_t e;
            CUDA_OK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            ctx->sync_events.push_back(e);
        }
        cudaEvent_t ev_start = ctx->sync_events[0], ev_tail = ctx->sync_events[1];
        // the staging area may still be in use by earlier work on the main stream
        CUDA_OK(cudaEventRecord(ev_start, ctx->stream));
        CUDA_OK(cudaStreamWaitEvent(ctx->copy_in, ev_start, 0));
        CUDA_OK(cudaStreamWaitEvent(ctx->copy_out, ev_start, 0));
        for (uint32_t j = 0; j < n_chunks; ++j) {
            const uint32_t a = j * chunk, m = std::min(chunk, n - a);
            CUDA_OK(cudaMemcpy2DAsync(x_dev + (uint64_t)a * row, row * sizeof(float), x_host + (uint64_t)a * ld_x,
                                      ld_x * sizeof(float), row_bytes, m, cudaMemcpyHostToDevice, ctx->copy_in));
            CUDA_OK(cudaEventRecord(ctx->sync_events[2 + 2 * j], ctx->copy_in));
        }
        ctx->ws_bytes = st.left;
        int rc = EDEN_OK;
        for (uint32_t j = 0; j < n_chunks && rc == EDEN_OK; ++j) {
            const uint32_t a = j * chunk, m = std::min(chunk, n - a);
            if (cudaStreamWaitEvent(ctx->stream, ctx->sync_events[2 + 2 * j], 0) != cudaSuccess) { rc = EDEN_ERR_CUDA; break; }
            rc = eden_encode(ctx, x_dev + (uint64_t)a * row, row, d, m, bits + a, seeds + a,
                             codes_dev.data() + a, scales_dev + a);
            if (rc) break;
            if (cudaEventRecord(ctx->sync_events[3 + 2 * j], ctx->stream) != cudaSuccess ||
                cudaStreamWaitEvent(ctx->copy_out, ctx->sync_events[3 + 2 * j], 0) != cudaSuccess) { rc = EDEN_ERR_CUDA; break; }
            for (uint32_t c = a; c < a + m; ++c)
                if (cudaMemcpyAsync(codes_host[c], codes_dev[c], eden_code_bytes(d, bits[c]),
                                    cudaMemcpyDeviceToHost, ctx->copy_out) != cudaSuccess) { rc = EDEN_ERR_CUDA; break; }
        }
        ctx->ws_bytes = saved;
        // join the side streams back into the main stream whatever happened
        cudaEventRecord(ev_tail, ctx->copy_out);
        cudaStreamWaitEvent(ctx->stream, ev_tail, 0);
        cudaEventRecord(ev_start, ctx->copy_in);
        cudaStreamWaitEvent(ctx->stream, ev_start, 0);
        if (rc) { cudaStreamSynchronize(ctx->stream); return rc; }
        CUDA_OK(cudaMemcpyAsync(scales_host, scales_dev, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
        CUDA_OK(cudaStreamSynchronize(ctx->stream));
        return EDEN_OK;
    }
    CUDA_OK(cudaMemcpy2DAsync(x_dev, row * sizeof(float), x_host, ld_x * sizeof(float),
                              d * sizeof(float), n, cudaMemcpyHostToDevice, ctx->stream));
    ctx->ws_bytes = st.left;
    const int rc = eden_encode(ctx, x_dev, row, d, n, bits, seeds, codes_dev.data(), scales_dev);
    ctx->ws_bytes = saved;
    if (rc) return rc;
    for (uint32_t c = 0; c < n; ++c)
        CUDA_OK(cudaMemcpyAsync(codes_host[c], codes_dev[c], eden_code_bytes(d, bits[c]),
                                cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_OK(cudaMemcpyAsync(scales_host, scales_dev, n * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
    return EDEN_OK;
}

extern "C" int eden_mean_host(eden_ctx* ctx, const uint8_t* const* codes_host, const float* scales_host,
                              const double* bits, const uint64_t* seeds,
                              const uint32_t* const* recv_masks_host,
                              uint64_t d, uint32_t n, float* mean_host)
{
    if (!ctx || !codes_host || !scales_host || !bits || !seeds || !mean_host || d == 0 || n == 0)
        return EDEN_ERR_INVALID_ARG;
    for (uint32_t c = 0; c < n; ++c)
        if (eden_code_width(bits[c]) == 0) return EDEN_ERR_UNSUPPORTED_BITS;
    CUDA_OK(cudaSetDevice(ctx->device));
    Staging st{ctx->ws, ctx->ws_bytes};
    float* mean_dev = (float*)st.take(d * sizeof(float));
    float* scales_dev = (float*)st.take(n * sizeof(float));
    if (!mean_dev || !scales_dev) return EDEN_ERR_WORKSPACE;
    std::vector<const uint8_t*> codes_dev(n);
    std::vector<const uint32_t*> masks_dev(n, nullptr);
    for (uint32_t c = 0; c < n; ++c) {
        const uint64_t cb = eden_code_bytes(d, bits[c]);
        uint8_t* p = (uint8_t*)st.take(cb);
        if (!p) return EDEN_ERR_WORKSPACE;
        CUDA_OK(cudaMemcpyAsync(p, codes_host[c], cb, cudaMemcpyHostToDevice, ctx->stream));
        codes_dev[c] = p;
        if (recv_masks_host && recv_masks_host[c]) {
            const uint64_t mb = eden_recv_mask_words(d, bits[c]) * 4;
            uint32_t* m = (uint32_t*)st.take(mb);
            if (!m) return EDEN_ERR_WORKSPACE;
            CUDA_OK(cudaMemcpyAsync(m, recv_masks_host[c], mb, cudaMemcpyHostToDevice, ctx->stream));
            masks_dev[c] = m;
        }
    }
    CUDA_OK(cudaMemcpyAsync(scales_dev, scales_host, n * sizeof(float), cudaMemcpyHostToDevice, ctx->stream));
    const uint64_t saved = ctx->ws_bytes;
    ctx->ws_bytes = st.left;
    const int rc = eden_mean(ctx, codes_dev.data(), scales_dev, bits, seeds,
                             recv_masks_host ? masks_dev.data() : nullptr, d, n, mean_dev);
    ctx->ws_bytes = saved;
    if (rc) return rc;
    CUDA_OK(cudaMemcpyAsync(mean_host, mean_dev, d * sizeof(float), cudaMemcpyDeviceToHost, ctx->stream));
    CUDA_OK(cudaStreamSynchronize(ctx->stream));
    return EDEN_OK;
}

// ------------------------------------------------------------------------------------
// Sparsification mask without any allocation or context.
//
// Some callers cannot hand this library a workspace because they cannot allocate device
// memory at the moment they need the mask: a receiver thread inside a host application
// whose caching allocator has already claimed the whole card (a raw cudaMalloc fails
// there), a service that freezes its memory map after start-up, or a latency-critical
// loop that must not take the device-wide synchronisation an allocation implies.  For
// them the scratch of the mask selection lives in the array below, which every GPU that
// loads this library carries until the process exits.
// ------------------------------------------------------------------------------------
namespace {

constexpr uint64_t kNoallocMaxDim = EDEN_NOALLOC_MAX_DIM;
constexpr uint64_t kNoallocSelOff = 0;
constexpr uint64_t kNoallocHistOff = 256;
constexpr uint64_t kNoallocChunkOff = kNoallocHistOff + kHistBytes;
constexpr uint64_t kNoallocBytes =
    kNoallocChunkOff + (kNoallocMaxDim / kSelChunk) * sizeof(unsigned long long);

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoallocBytes];

// In host code the name g_noalloc_scratch is only a handle: the device address has to be
// asked for, once per device, with that device current.
constexpr int kNoallocMaxDevices = 64;
std::mutex g_noalloc_mutex;
unsigned char* g_noalloc_ptr[kNoallocMaxDevices];

int noalloc_scratch(int device, unsigned char** out)
{
    if (device < 0 || device >= kNoallocMaxDevices) return EDEN_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return EDEN_ERR_CUDA;
        g_noalloc_ptr[device] = (unsigned char*)p;
    }
    *out = g_noalloc_ptr[device];
    return EDEN_OK;
}

// Makes `device` current for the life of the object and puts the caller's device back.
struct DeviceScope {
    int previous;
    bool changed;
    cudaError_t status;
    explicit DeviceScope(int device) : previous(-1), changed(false), status(cudaGetDevice(&previous))
    {
        if (status == cudaSuccess && previous != device) {
            status = cudaSetDevice(device);
            changed = status == cudaSuccess;
        }
    }
    ~DeviceScope()
    {
        if (changed) cudaSetDevice(previous);
    }
};

}  // namespace

extern "C" int eden_sparsification_mask_noalloc(int cuda_device, void* cuda_stream, uint64_t seed,
                                                uint64_t d, double bits, uint32_t* mask_bits)
{
    if (!mask_bits || d == 0 || !(bits > 0.0) || !(bits < 1.0)) return EDEN_ERR_INVALID_ARG;
    if (d > kNoallocMaxDim) return EDEN_ERR_TOO_LARGE;
    const DeviceScope scope(cuda_device);          // the caller's current device is put back on return
    CUDA_OK(scope.status);
    unsigned char* base = nullptr;
    const int rc = noalloc_scratch(cuda_device, &base);
    if (rc) return rc;
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    MaskSelect* sel = (MaskSelect*)(base + kNoallocSelOff);
    uint32_t* hist = (uint32_t*)(base + kNoallocHistOff);
    unsigned long long* chunks = (unsigned long long*)(base + kNoallocChunkOff);
    const uint64_t k = eden_kept_count(d, bits);
    const unsigned grid = (unsigned)(((d + 3) / 4 + kSelThreads - 1) / kSelThreads);
    // the array keeps the previous call's contents: the histograms must start at zero;
    // everything else is overwritten before it is read
    CUDA_OK(cudaMemsetAsync(hist, 0, kHistBytes, stream));
    k_sel_hist<<<grid, kSelThreads, 0, stream>>>(seed, d, 0, sel, hist);
    k_sel_find<<<1, 1024, 0, stream>>>(hist, k, 0, sel);
    k_sel_hist<<<grid, kSelThreads, 0, stream>>>(seed, d, 1, sel, hist + 65536);
    k_sel_find<<<1, 1024, 0, stream>>>(hist + 65536, k, 1, sel);
    k_sel_chunk_count<<<grid, kSelThreads, 0, stream>>>(seed, d, sel, chunks);
    k_sel_chunk_scan<<<1, 1024, 0, stream>>>(chunks, (uint64_t)grid);
    k_sel_apply<SEL_MASK_BITS><<<grid, kSelThreads, 0, stream>>>(
        seed, d, sel, chunks, (const float*)nullptr, (float*)nullptr, mask_bits);
    if (cudaGetLastError() != cudaSuccess) return EDEN_ERR_CUDA;
    return EDEN_OK;
}
