// C ABI of libelsa: host-side validation, dispatch and error reporting.  No kernel lives here.

#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "elsa_internal.h"

namespace elsa {

static thread_local char g_error[512] = "";
static std::atomic<unsigned long long> g_launches{0};
static std::atomic<int> g_variant{(int)ELSA_VARIANT_AUTO};
static std::atomic<bool> g_grouping{true};

namespace {
struct ProfileRecord {
    int kernel, layer;
    cudaEvent_t start, stop;
};
std::atomic<bool> g_profile_on{false};
std::mutex g_profile_mutex;
std::vector<ProfileRecord> g_profile;
thread_local int g_profile_layer = -1;
}  // namespace

void set_profile_layer(int layer) { g_profile_layer = layer; }

ProfileScope::ProfileScope(int kernel, cudaStream_t stream) : slot_(-1), stream_(stream)
{
    if (!g_profile_on.load(std::memory_order_relaxed)) return;
    ProfileRecord r;
    r.kernel = kernel;
    r.layer = g_profile_layer;
    if (cudaEventCreate(&r.start) != cudaSuccess) { cudaGetLastError(); return; }
    if (cudaEventCreate(&r.stop) != cudaSuccess) { cudaGetLastError(); cudaEventDestroy(r.start); return; }
    cudaEventRecord(r.start, stream);
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    g_profile.push_back(r);
    slot_ = (int)g_profile.size() - 1;
}

ProfileScope::~ProfileScope()
{
    if (slot_ < 0) return;
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    if (slot_ < (int)g_profile.size()) cudaEventRecord(g_profile[slot_].stop, stream_);
}

elsa_status fail(elsa_status st, const char* fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
    return st;
}

elsa_status launched(const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ELSA_ERR_CUDA, "launch of %s failed: %s", what, cudaGetErrorString(e));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return ELSA_OK;
}

elsa_status device_info(DeviceInfo* info)
{
    static DeviceInfo cache[64];
    static std::atomic<bool> have[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaError_t e = cudaGetLastError();
        return fail(ELSA_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    }
    const int slot = dev & 63;
    if (!have[slot].load(std::memory_order_acquire)) {
        DeviceInfo d;
        d.device = dev;
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) goto bad;
        d.sm_count = v;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) goto bad;
        d.cc_major = v;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) goto bad;
        d.smem_optin = (size_t)v;
        cache[slot] = d;
        have[slot].store(true, std::memory_order_release);
    }
    *info = cache[slot];
    if (info->cc_major != 10)
        return fail(ELSA_ERR_ARCH, "device %d has compute capability %d.x; this library is built for 10.x only",
                    dev, info->cc_major);
    return ELSA_OK;
bad:
    cudaError_t e = cudaGetLastError();
    return fail(ELSA_ERR_CUDA, "cudaDeviceGetAttribute: %s", cudaGetErrorString(e));
}

namespace {

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

elsa_status check_level(int out, int in, int N, int M, int dtype)
{
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return fail(ELSA_ERR_DTYPE, "dtype %d is neither ELSA_F16 nor ELSA_BF16", dtype);
    if (out <= 0 || in <= 0) return fail(ELSA_ERR_SHAPE, "non-positive dimension (out=%d, in=%d)", out, in);
    if (index_bits(M) < 0 || N < 1 || N > M) return fail(ELSA_ERR_NM, "unsupported level %d:%d (M in {4, 8, 16}, 1 <= N <= M)", N, M);
    if (in % M != 0) return fail(ELSA_ERR_SHAPE, "in=%d is not a multiple of M=%d", in, M);
    if (in % 8 != 0 || out % 8 != 0) return fail(ELSA_ERR_ALIGN, "in=%d and out=%d must be multiples of 8 (16-byte row pitch)", in, out);
    return ELSA_OK;
}

elsa_status check_linear(const void* X, int rows, const void* vals, const uint32_t* idx, const void* bias,
                         int out, int in, int N, int M, int dtype, const void* Y, const void* workspace,
                         size_t workspace_bytes)
{
    if (!X || !vals || !Y) return fail(ELSA_ERR_NULL, "X, vals and Y must not be NULL");
    elsa_status st = check_level(out, in, N, M, dtype);
    if (st != ELSA_OK) return st;
    if (rows <= 0) return fail(ELSA_ERR_SHAPE, "non-positive rows=%d", rows);
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(X) || !aligned16(vals) || !aligned16(Y) || (idx && !aligned16(idx)) ||
        (bias && !aligned16(bias)))
        return fail(ELSA_ERR_ALIGN, "X, vals, idx, bias and Y must be 16-byte aligned");
    const size_t need = elsa_workspace_bytes(rows, in, out, N, M, (elsa_dtype)dtype);
    if (need) {
        if (!workspace || workspace_bytes < need)
            return fail(ELSA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace ? workspace_bytes : (size_t)0);
        if (((uintptr_t)workspace & 255u) != 0) return fail(ELSA_ERR_ALIGN, "workspace must be 256-byte aligned");
    }
    return ELSA_OK;
}

// Side stream of elsa_vit_linears (weight images beside the dense layers), created once per device.
struct SidePipe {
    cudaStream_t stream;
    cudaEvent_t fork, join;
    bool ready;
};
SidePipe g_side[64];
std::mutex g_side_mutex;

elsa_status side_pipe(int device, SidePipe** pipe)
{
    std::lock_guard<std::mutex> lock(g_side_mutex);
    SidePipe& p = g_side[device & 63];
    if (!p.ready) {
        const bool ok = cudaStreamCreateWithFlags(&p.stream, cudaStreamNonBlocking) == cudaSuccess &&
                        cudaEventCreateWithFlags(&p.fork, cudaEventDisableTiming) == cudaSuccess &&
                        cudaEventCreateWithFlags(&p.join, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "creating the image stream: %s", cudaGetErrorString(e));
        }
        p.ready = true;
    }
    *pipe = &p;
    return ELSA_OK;
}

enum LinearKind { KIND_SIMT, KIND_DENSE_ONE, KIND_DENSE_PAIR, KIND_SPARSE_ONE, KIND_SPARSE_PAIR, KIND_SPARSE_WS, KIND_SPARSE_ST };

// Form of the 2-of-4 weight image each sparse kernel reads.
int sp24_layout_of(LinearKind kind)
{
    return kind == KIND_SPARSE_WS ? SP24_PERMUTED : kind == KIND_SPARSE_ST ? SP24_TILED : SP24_ROWS;
}

// Which kernel a layer runs on.  AUTO is the product rule; a forced variant is honoured where it applies.
elsa_status pick_kind(int rows, int out, int in, int N, int M, int sm_count, LinearKind* kind)
{
    const int variant = g_variant.load(std::memory_order_relaxed);
    const bool sparse_ok = N != M && linear_tc_sparse_suits(in, N);
    switch (variant) {
    case ELSA_VARIANT_SIMT: *kind = KIND_SIMT; return ELSA_OK;
    case ELSA_VARIANT_TC_DENSE: *kind = KIND_DENSE_ONE; return ELSA_OK;
    case ELSA_VARIANT_TC_PAIR: *kind = KIND_DENSE_PAIR; return ELSA_OK;
    case ELSA_VARIANT_TC_SPARSE:
    case ELSA_VARIANT_TC_SPARSE_PAIR:
        if (!sparse_ok)
            return fail(ELSA_ERR_NM, "the sparse-MMA variant needs N <= 2 < M and in %% 16 == 0 (got %d:%d, in=%d)", N, M, in);
        *kind = variant == ELSA_VARIANT_TC_SPARSE ? KIND_SPARSE_ONE : KIND_SPARSE_PAIR;
        return ELSA_OK;
    case ELSA_VARIANT_TC_SPARSE_WS:
        if (N == M || !linear_tc_sparse_ws_suits(in, out, N, sm_count))
            return fail(ELSA_ERR_NM, "the weight-stationary sparse variant needs N <= 2 < M, in %% 128 == 0 and in <= 1024 "
                        "(got %d:%d, in=%d)", N, M, in);
        *kind = KIND_SPARSE_WS;
        return ELSA_OK;
    case ELSA_VARIANT_TC_SPARSE_ST:
        if (N == M || !linear_tc_sparse_st_suits(in, N))
            return fail(ELSA_ERR_NM, "the streaming sparse variant needs N <= 2 < M and in %% 128 == 0 (got %d:%d, in=%d)", N, M, in);
        *kind = KIND_SPARSE_ST;
        return ELSA_OK;
    default: break;
    }
    // Levels with N <= 2 fit the 2:4 sparse MMA.  Measured on B200 it beats the dense-rate kernels from K = 256
    // up once there are enough tiles to fill the CTA pairs; K = 128 layers are pure streaming problems and
    // stay on the dense-rate path.
    if (sparse_ok && in >= 256 && (long long)((rows + 223) / 224) * ((out + 255) / 256) >= sm_count / 4) {
        // With the weight block resident in tensor memory the activations are the only shared-memory
        // traffic: every layer whose reduction fits (in <= 896) and that has at least two blocks of 256
        // features goes there.
        const bool ws = linear_tc_sparse_ws_suits(in, out, N, sm_count) && in <= 896 && out >= 512 &&
                        rows >= 256 * (sm_count / 2) / ((out + 255) / 256);
        // Longer reductions do not fit tensor memory whole: the weight streams through it chunk by chunk, which
        // still keeps it out of shared memory (measured against staging it there for every row tile).
        const bool st = !ws && in > 768 && linear_tc_sparse_st_suits(in, N);
        *kind = ws ? KIND_SPARSE_WS : st ? KIND_SPARSE_ST : KIND_SPARSE_PAIR;
    }
    else
        *kind = linear_tc_pair_suits(rows, out, sm_count) ? KIND_DENSE_PAIR : KIND_DENSE_ONE;
    return ELSA_OK;
}

// After validation: enqueue one layer.
elsa_status run_linear(const void* X, int rows, const void* vals, const uint32_t* idx, const void* bias, int out,
                       int in, int N, int M, elsa_dtype dtype, void* Y, void* workspace, uint32_t* dev_status,
                       cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    LinearKind kind;
    if ((st = pick_kind(rows, out, in, N, M, dev.sm_count, &kind)) != ELSA_OK) return st;
    if (kind == KIND_SIMT)
        return launch_linear_simt((const uint16_t*)X, rows, (const uint16_t*)vals, idx, (const uint16_t*)bias, out,
                                  in, N, M, dtype, (uint16_t*)Y, stream);
    if (kind == KIND_SPARSE_ONE)
        return launch_linear_tc_sparse((const uint16_t*)X, rows, (const uint16_t*)vals, idx, (const uint16_t*)bias, out,
                                       in, N, M, dtype, (uint16_t*)Y, workspace, dev_status, stream);
    if (kind == KIND_SPARSE_PAIR)
        return launch_linear_tc_sparse_pair((const uint16_t*)X, rows, (const uint16_t*)vals, idx, (const uint16_t*)bias,
                                            out, in, N, M, dtype, (uint16_t*)Y, workspace, dev_status, stream);
    if (kind == KIND_SPARSE_WS)
        return launch_linear_tc_sparse_ws((const uint16_t*)X, rows, (const uint16_t*)vals, idx, (const uint16_t*)bias,
                                          out, in, N, M, dtype, (uint16_t*)Y, workspace, dev_status, stream);
    if (kind == KIND_SPARSE_ST)
        return launch_linear_tc_sparse_st((const uint16_t*)X, rows, (const uint16_t*)vals, idx, (const uint16_t*)bias,
                                          out, in, N, M, dtype, (uint16_t*)Y, workspace, dev_status, stream);
    // Dense-rate path.  The dense level multiplies the stored values as they are; every other level first
    // rebuilds the weight image the MMA reads, in the caller's scratch.
    const uint16_t* Wd = (const uint16_t*)vals;
    if (N != M) {
        if ((st = launch_unpack((const uint16_t*)vals, idx, out, in, N, M, (uint16_t*)workspace, stream)) != ELSA_OK)
            return st;
        Wd = (const uint16_t*)workspace;
    }
    if (kind == KIND_DENSE_PAIR)
        return launch_linear_tc_pair((const uint16_t*)X, rows, Wd, (const uint16_t*)bias, out, in, dtype,
                                     (uint16_t*)Y, dev_status, stream);
    return launch_linear_tc_dense((const uint16_t*)X, rows, Wd, (const uint16_t*)bias, out, in, dtype,
                                  (uint16_t*)Y, dev_status, stream);
}

}  // namespace
}  // namespace elsa

using namespace elsa;

extern "C" {

size_t elsa_nm_values_bytes(int out, int in, int N, int M, elsa_dtype dtype)
{
    if (out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return 0;
    return (size_t)out * values_per_row(in, N, M) * 2;
}

size_t elsa_nm_index_bytes(int out, int in, int N, int M)
{
    if (out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    return (size_t)out * index_words_per_row(in, N, M) * 4;
}

size_t elsa_workspace_bytes(int rows, int in, int out, int N, int M, elsa_dtype dtype)
{
    (void)rows;
    if (out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return 0;
    if (N == M) return 0;                              // the dense level needs no weight image
    size_t need = round_up((size_t)out * (size_t)in * 2, 256);  // dense image of the masked weight
    if (linear_tc_sparse_suits(in, N)) {                          // or its 2-of-4 image + metadata
        const size_t sp = round_up(linear_tc_sparse_workspace(out, in), 256);
        if (sp > need) need = sp;
    }
    return need;
}

elsa_status elsa_nm_compress(const void* W, int out, int in, int N, int M, elsa_dtype dtype, void* vals,
                             uint32_t* idx, void* stream)
{
    if (!W || !vals) return fail(ELSA_ERR_NULL, "W and vals must not be NULL");
    elsa_status st = check_level(out, in, N, M, dtype);
    if (st != ELSA_OK) return st;
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(W) || !aligned16(vals) || (idx && !aligned16(idx)))
        return fail(ELSA_ERR_ALIGN, "W, vals and idx must be 16-byte aligned");
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    return launch_compress((const uint16_t*)W, out, in, N, M, (uint16_t*)vals, N == M ? nullptr : idx,
                           (cudaStream_t)stream);
}

elsa_status elsa_nm_unpack(const void* vals, const uint32_t* idx, int out, int in, int N, int M, elsa_dtype dtype,
                           void* W_masked, void* stream)
{
    if (!vals || !W_masked) return fail(ELSA_ERR_NULL, "vals and W_masked must not be NULL");
    elsa_status st = check_level(out, in, N, M, dtype);
    if (st != ELSA_OK) return st;
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(vals) || !aligned16(W_masked) || (idx && !aligned16(idx)))
        return fail(ELSA_ERR_ALIGN, "vals, idx and W_masked must be 16-byte aligned");
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    return launch_unpack((const uint16_t*)vals, N == M ? nullptr : idx, out, in, N, M, (uint16_t*)W_masked,
                         (cudaStream_t)stream);
}

elsa_status elsa_nm_linear(const void* X, int rows, const void* vals, const uint32_t* idx, const void* bias,
                           int out, int in, int N, int M, elsa_dtype dtype, void* Y, void* workspace,
                           size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    elsa_status st = check_linear(X, rows, vals, idx, bias, out, in, N, M, dtype, Y, workspace, workspace_bytes);
    if (st != ELSA_OK) return st;
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    return run_linear(X, rows, vals, N == M ? nullptr : idx, bias, out, in, N, M, dtype, Y, workspace, dev_status,
                      (cudaStream_t)stream);
}

elsa_status elsa_nm_compress_levels(const void* W, int out, int in, int M, const int* N_list, int n_levels,
                                    elsa_dtype dtype, void* const* vals, uint32_t* const* idx, void* stream)
{
    if (!W || !N_list || !vals || !idx) return fail(ELSA_ERR_NULL, "W, N_list, vals and idx must not be NULL");
    if (n_levels < 1 || n_levels > kMaxLevels)
        return fail(ELSA_ERR_SHAPE, "n_levels=%d is outside 1..%d", n_levels, kMaxLevels);
    if (!aligned16(W)) return fail(ELSA_ERR_ALIGN, "W must be 16-byte aligned");
    LevelTable t;
    t.n = n_levels;
    for (int l = 0; l < n_levels; ++l) {
        elsa_status st = check_level(out, in, N_list[l], M, dtype);
        if (st == ELSA_OK && !vals[l]) st = fail(ELSA_ERR_NULL, "vals must not be NULL");
        if (st == ELSA_OK && N_list[l] != M && !idx[l]) st = fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
        if (st == ELSA_OK && (!aligned16(vals[l]) || (idx[l] && !aligned16(idx[l]))))
            st = fail(ELSA_ERR_ALIGN, "vals and idx must be 16-byte aligned");
        if (st != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "level %d: %s", l, msg);
        }
        t.N[l] = N_list[l];
        t.vals[l] = (uint16_t*)vals[l];
        t.idx[l] = N_list[l] == M ? nullptr : idx[l];
    }
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    return launch_compress_levels((const uint16_t*)W, out, in, M, t, (cudaStream_t)stream);
}

elsa_status elsa_nm_linear_masked(const void* X, int rows, const void* W_sup, const void* bias, int out, int in,
                                  int N, int M, elsa_dtype dtype, void* Y, void* workspace, size_t workspace_bytes,
                                  uint32_t* dev_status, void* stream_)
{
    // the dense weight takes the place of vals in the checks (same alignment rules), no index words
    uint32_t* no_idx = N == M ? nullptr : (uint32_t*)W_sup;
    elsa_status st = check_linear(X, rows, W_sup, no_idx, bias, out, in, N, M, dtype, Y, workspace, workspace_bytes);
    if (st != ELSA_OK) return st;
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    LinearKind kind;
    if ((st = pick_kind(rows, out, in, N, M, dev.sm_count, &kind)) != ELSA_OK) return st;
    if (kind == KIND_SIMT || kind == KIND_SPARSE_ONE)
        return fail(ELSA_ERR_NM, "the forced variant has no mask-on-load form");
    if (kind == KIND_SPARSE_PAIR || kind == KIND_SPARSE_WS || kind == KIND_SPARSE_ST) {
        uint8_t* meta = (uint8_t*)workspace + sp24_meta_offset(out, in);
        if ((st = launch_dense_to_sp24((const uint16_t*)W_sup, out, in, N, M, 128, sp24_layout_of(kind), (uint16_t*)workspace, meta,
                                       stream)) != ELSA_OK)
            return st;
        SparseJob job;
        job.X = (const uint16_t*)X; job.bias = (const uint16_t*)bias; job.Y = (uint16_t*)Y; job.workspace = workspace;
        job.rows = rows; job.in = in; job.out = out;
        return kind == KIND_SPARSE_WS   ? launch_linear_tc_sparse_ws_group(&job, 1, dtype, dev_status, stream)
               : kind == KIND_SPARSE_ST ? launch_linear_tc_sparse_st_group(&job, 1, dtype, dev_status, stream)
                                        : launch_linear_tc_sparse_pair_group(&job, 1, dtype, dev_status, stream);
    }
    const uint16_t* Wd = (const uint16_t*)W_sup;     // the dense level multiplies the shared weight as it is
    if (N != M) {
        if ((st = launch_mask((const uint16_t*)W_sup, out, in, N, M, (uint16_t*)workspace, stream)) != ELSA_OK) return st;
        Wd = (const uint16_t*)workspace;
    }
    if (kind == KIND_DENSE_PAIR)
        return launch_linear_tc_pair((const uint16_t*)X, rows, Wd, (const uint16_t*)bias, out, in, dtype, (uint16_t*)Y,
                                     dev_status, stream);
    return launch_linear_tc_dense((const uint16_t*)X, rows, Wd, (const uint16_t*)bias, out, in, dtype, (uint16_t*)Y,
                                  dev_status, stream);
}

elsa_status elsa_vit_compress(const elsa_weight* w, int n_weights, elsa_dtype dtype, void* stream)
{
    if (!w) return fail(ELSA_ERR_NULL, "w must not be NULL");
    if (n_weights <= 0) return fail(ELSA_ERR_SHAPE, "non-positive n_weights=%d", n_weights);
    for (int i = 0; i < n_weights; ++i) {
        const elsa_weight& c = w[i];
        elsa_status st = ELSA_OK;
        if (!c.W || !c.vals) st = fail(ELSA_ERR_NULL, "W and vals must not be NULL");
        else if ((st = check_level(c.out, c.in, c.N, c.M, dtype)) != ELSA_OK) {}
        else if (c.N != c.M && !c.idx) st = fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
        else if (!aligned16(c.W) || !aligned16(c.vals) || (c.idx && !aligned16(c.idx)))
            st = fail(ELSA_ERR_ALIGN, "W, vals and idx must be 16-byte aligned");
        if (st != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "weight %d: %s", i, msg);
        }
    }
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    static BatchTable table;              // host staging of the kernel parameters
    static std::mutex table_mutex;
    std::lock_guard<std::mutex> lock(table_mutex);
    table.n = 0;
    table.total_units = 0;
    for (int i = 0; i < n_weights; ++i) {
        const elsa_weight& c = w[i];
        batch_add_compress(&table, (const uint16_t*)c.W, c.out, c.in, c.N, c.M, (uint16_t*)c.vals,
                           c.N == c.M ? nullptr : c.idx);
        if (table.n == kBatchMax || i == n_weights - 1) {
            if ((st = launch_compress_batch(table, (cudaStream_t)stream)) != ELSA_OK) return st;
            table.n = 0;
            table.total_units = 0;
        }
    }
    return ELSA_OK;
}

size_t elsa_vit_workspace_bytes(const elsa_layer* cfg, int n_layers, elsa_dtype dtype)
{
    // one region per layer, so that every weight image can be built before the grouped launches
    size_t need = 0;
    if (!cfg) return 0;
    for (int l = 0; l < n_layers; ++l)
        need += round_up(elsa_workspace_bytes(cfg[l].rows, cfg[l].in, cfg[l].out, cfg[l].N, cfg[l].M, dtype), 256);
    return need;
}

elsa_status elsa_vit_linears(const elsa_layer* cfg, int n_layers, elsa_dtype dtype, void* workspace,
                             size_t workspace_bytes, uint32_t* dev_status, void* stream_)
{
    if (!cfg) return fail(ELSA_ERR_NULL, "cfg must not be NULL");
    if (n_layers <= 0) return fail(ELSA_ERR_SHAPE, "non-positive n_layers=%d", n_layers);
    for (int l = 0; l < n_layers; ++l) {
        const elsa_layer& c = cfg[l];
        elsa_status st = check_linear(c.X, c.rows, c.vals, c.idx, c.bias, c.out, c.in, c.N, c.M, dtype, c.Y,
                                      workspace, workspace_bytes);
        if (st != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "layer %d: %s", l, msg);
        }
    }
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    auto layer_fail = [](elsa_status code, int l) {
        set_profile_layer(-1);
        char msg[400];
        snprintf(msg, sizeof msg, "%s", elsa_last_error());
        return fail(code, "layer %d: %s", l, msg);
    };

    // With one scratch region per layer (elsa_vit_workspace_bytes) all weight images are built first and the
    // layers of each kernel family share persistent launches: the layers of a table do not depend on one
    // another, so their tiles may interleave.  With less scratch (at least the largest layer's, which
    // validation has checked) the layers run one after the other through the same region.
    const bool grouped = g_grouping.load(std::memory_order_relaxed) &&
                         g_variant.load(std::memory_order_relaxed) == ELSA_VARIANT_AUTO &&
                         workspace_bytes >= elsa_vit_workspace_bytes(cfg, n_layers, dtype);
    if (!grouped) {
        for (int l = 0; l < n_layers; ++l) {
            const elsa_layer& c = cfg[l];
            set_profile_layer(l);
            st = run_linear(c.X, c.rows, c.vals, c.N == c.M ? nullptr : c.idx, c.bias, c.out, c.in, c.N, c.M, dtype,
                            c.Y, workspace, dev_status, stream);
            if (st != ELSA_OK) return layer_fail(st, l);
        }
        set_profile_layer(-1);
        return ELSA_OK;
    }

    // The weight images are built on a side stream while the dense layers, which need none, already run on
    // the caller's: the image kernel is a small streaming kernel whose blocks fit beside the persistent GEMM's
    // one CTA per SM.  Everything else waits for the images.
    SidePipe* side = nullptr;
    if ((st = side_pipe(dev.device, &side)) != ELSA_OK) return st;
    std::vector<LinearKind> kind(n_layers);
    std::vector<uint8_t*> region(n_layers);
    size_t off = 0;
    for (int l = 0; l < n_layers; ++l) {
        const elsa_layer& c = cfg[l];
        if ((st = pick_kind(c.rows, c.out, c.in, c.N, c.M, dev.sm_count, &kind[l])) != ELSA_OK) return layer_fail(st, l);
        region[l] = (uint8_t*)workspace + off;
        off += round_up(elsa_workspace_bytes(c.rows, c.in, c.out, c.N, c.M, dtype), 256);
    }
    // dense-rate layers that multiply the stored values as they are (N = M), on CTA pairs, in groups: launched
    // first, the weight images are built beside them
    bool forked = false;
    {
        std::vector<PairJob> jobs;
        for (int l = 0; l <= n_layers; ++l) {
            if (l < n_layers && kind[l] == KIND_DENSE_PAIR && cfg[l].N == cfg[l].M) {
                const elsa_layer& c = cfg[l];
                PairJob j;
                j.X = (const uint16_t*)c.X; j.bias = (const uint16_t*)c.bias; j.Y = (uint16_t*)c.Y;
                j.Wd = (const uint16_t*)c.vals;
                j.rows = c.rows; j.in = c.in; j.out = c.out;
                jobs.push_back(j);
            }
            if (!jobs.empty() && (l == n_layers || (int)jobs.size() == linear_tc_pair_group_max())) {
                if (!forked) {
                    // the side stream starts where the caller's stream stands now (after the compress kernels)
                    cudaError_t e = cudaEventRecord(side->fork, stream);
                    if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
                    if (e != cudaSuccess) { cudaGetLastError(); return fail(ELSA_ERR_CUDA, "forking the image stream: %s", cudaGetErrorString(e)); }
                    forked = true;
                }
                if ((st = launch_linear_tc_pair_group(jobs.data(), (int)jobs.size(), dtype, dev_status, stream)) != ELSA_OK)
                    return st;
                jobs.clear();
            }
        }
    }
    cudaStream_t image_stream = forked ? side->stream : stream;
    // weight images of all layers, one launch per 256 layers
    {
        static BatchTable table;          // host staging of the kernel parameters
        static std::mutex table_mutex;
        std::lock_guard<std::mutex> lock(table_mutex);
        table.n = 0;
        table.total_units = 0;
        for (int l = 0; l < n_layers; ++l) {
            const elsa_layer& c = cfg[l];
            if (c.N != c.M) {
                if (kind[l] == KIND_SPARSE_PAIR || kind[l] == KIND_SPARSE_WS || kind[l] == KIND_SPARSE_ST) {
                    uint8_t* meta = region[l] + sp24_meta_offset(c.out, c.in);
                    batch_add_to_sp24(&table, (const uint16_t*)c.vals, c.idx, c.out, c.in, c.N, c.M, 128,
                                      sp24_layout_of(kind[l]), (uint16_t*)region[l], meta);
                } else {
                    batch_add_unpack(&table, (const uint16_t*)c.vals, c.idx, c.out, c.in, c.N, c.M, (uint16_t*)region[l]);
                }
            }
            if (table.n == kBatchMax || (l == n_layers - 1 && table.n > 0)) {
                if ((st = launch_image_batch(table, image_stream)) != ELSA_OK) return st;
                table.n = 0;
                table.total_units = 0;
            }
        }
    }
    if (forked) {
        cudaError_t e = cudaEventRecord(side->join, side->stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, side->join, 0);
        if (e != cudaSuccess) { cudaGetLastError(); return fail(ELSA_ERR_CUDA, "joining the image stream: %s", cudaGetErrorString(e)); }
    }
    // sparse-rate layers, in groups
    {
        std::vector<SparseJob> jobs;
        for (int l = 0; l <= n_layers; ++l) {
            if (l < n_layers && kind[l] == KIND_SPARSE_PAIR) {
                const elsa_layer& c = cfg[l];
                SparseJob j;
                j.X = (const uint16_t*)c.X; j.bias = (const uint16_t*)c.bias; j.Y = (uint16_t*)c.Y;
                j.workspace = region[l]; j.rows = c.rows; j.in = c.in; j.out = c.out;
                jobs.push_back(j);
            }
            if (!jobs.empty() && (l == n_layers || (int)jobs.size() == linear_tc_sparse_pair_group_max())) {
                if ((st = launch_linear_tc_sparse_pair_group(jobs.data(), (int)jobs.size(), dtype, dev_status, stream)) != ELSA_OK)
                    return st;
                jobs.clear();
            }
        }
    }
    // sparse-rate layers whose weight block streams through tensor memory, in groups
    {
        std::vector<SparseJob> jobs;
        for (int l = 0; l <= n_layers; ++l) {
            if (l < n_layers && kind[l] == KIND_SPARSE_ST) {
                const elsa_layer& c = cfg[l];
                SparseJob j;
                j.X = (const uint16_t*)c.X; j.bias = (const uint16_t*)c.bias; j.Y = (uint16_t*)c.Y;
                j.workspace = region[l]; j.rows = c.rows; j.in = c.in; j.out = c.out;
                jobs.push_back(j);
            }
            if (!jobs.empty() && (l == n_layers || (int)jobs.size() == linear_tc_sparse_st_group_max())) {
                if ((st = launch_linear_tc_sparse_st_group(jobs.data(), (int)jobs.size(), dtype, dev_status, stream)) != ELSA_OK)
                    return st;
                jobs.clear();
            }
        }
    }
    // sparse-rate layers whose weight block fits tensor memory, in groups
    {
        std::vector<SparseJob> jobs;
        for (int l = 0; l <= n_layers; ++l) {
            if (l < n_layers && kind[l] == KIND_SPARSE_WS) {
                const elsa_layer& c = cfg[l];
                SparseJob j;
                j.X = (const uint16_t*)c.X; j.bias = (const uint16_t*)c.bias; j.Y = (uint16_t*)c.Y;
                j.workspace = region[l]; j.rows = c.rows; j.in = c.in; j.out = c.out;
                jobs.push_back(j);
            }
            if (!jobs.empty() && (l == n_layers || (int)jobs.size() == linear_tc_sparse_ws_group_max())) {
                if ((st = launch_linear_tc_sparse_ws_group(jobs.data(), (int)jobs.size(), dtype, dev_status, stream)) != ELSA_OK)
                    return st;
                jobs.clear();
            }
        }
    }
    // dense-rate layers that read a weight image (N < M), on CTA pairs, in groups
    {
        std::vector<PairJob> jobs;
        for (int l = 0; l <= n_layers; ++l) {
            if (l < n_layers && kind[l] == KIND_DENSE_PAIR && cfg[l].N != cfg[l].M) {
                const elsa_layer& c = cfg[l];
                PairJob j;
                j.X = (const uint16_t*)c.X; j.bias = (const uint16_t*)c.bias; j.Y = (uint16_t*)c.Y;
                j.Wd = c.N == c.M ? (const uint16_t*)c.vals : (const uint16_t*)region[l];
                j.rows = c.rows; j.in = c.in; j.out = c.out;
                jobs.push_back(j);
            }
            if (!jobs.empty() && (l == n_layers || (int)jobs.size() == linear_tc_pair_group_max())) {
                if ((st = launch_linear_tc_pair_group(jobs.data(), (int)jobs.size(), dtype, dev_status, stream)) != ELSA_OK)
                    return st;
                jobs.clear();
            }
        }
    }
    // small layers: one CTA per tile, one launch each
    for (int l = 0; l < n_layers; ++l) {
        if (kind[l] != KIND_DENSE_ONE) continue;
        const elsa_layer& c = cfg[l];
        set_profile_layer(l);
        const uint16_t* Wd = c.N == c.M ? (const uint16_t*)c.vals : (const uint16_t*)region[l];
        st = launch_linear_tc_dense((const uint16_t*)c.X, c.rows, Wd, (const uint16_t*)c.bias, c.out, c.in, dtype,
                                    (uint16_t*)c.Y, dev_status, stream);
        if (st != ELSA_OK) return layer_fail(st, l);
    }
    set_profile_layer(-1);
    return ELSA_OK;
}

// Device memory plan of the host-memory variant: two slots, used by alternate layers so that the
// copies of one layer overlap the kernels of its neighbours; each slot holds regions sized for the
// largest layer: X | Y | W | bias | vals | idx | linear workspace.
namespace {
struct HostPlan {
    size_t x, y, w, bias, vals, idx, ws, slot, total;
};

// Copy streams and ordering events of the host-memory variant, created once per device.
struct HostPipe {
    cudaStream_t in, out;
    cudaEvent_t start, in_done[2], compute_done[2], out_done[2];
    bool ready;
};
HostPipe g_pipe[64];
std::mutex g_pipe_mutex;

elsa_status host_pipe(int device, HostPipe** pipe)
{
    std::lock_guard<std::mutex> lock(g_pipe_mutex);
    HostPipe& p = g_pipe[device & 63];
    if (!p.ready) {
        bool ok = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&p.start, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; ok && i < 2; ++i)
            ok = cudaEventCreateWithFlags(&p.in_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.compute_done[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&p.out_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "creating the copy streams: %s", cudaGetErrorString(e));
        }
        p.ready = true;
    }
    *pipe = &p;
    return ELSA_OK;
}
bool host_plan(const elsa_host_layer* cfg, int n_layers, elsa_dtype dtype, HostPlan* plan)
{
    size_t mx = 0, my = 0, mw = 0, mb = 0, mv = 0, mi = 0, ms = 0;
    for (int l = 0; l < n_layers; ++l) {
        const elsa_host_layer& c = cfg[l];
        if (c.rows <= 0 || c.in <= 0 || c.out <= 0) return false;
        auto up = [](size_t& m, size_t v) { if (v > m) m = v; };
        up(mx, (size_t)c.rows * c.in * 2);
        up(my, (size_t)c.rows * c.out * 2);
        up(mw, (size_t)c.out * c.in * 2);
        up(mb, (size_t)c.out * 2);
        up(mv, elsa_nm_values_bytes(c.out, c.in, c.N, c.M, dtype));
        up(mi, elsa_nm_index_bytes(c.out, c.in, c.N, c.M));
        up(ms, elsa_workspace_bytes(c.rows, c.in, c.out, c.N, c.M, dtype));
    }
    size_t off = 0;
    plan->x = off; off += round_up(mx, 256);
    plan->y = off; off += round_up(my, 256);
    plan->w = off; off += round_up(mw, 256);
    plan->bias = off; off += round_up(mb, 256);
    plan->vals = off; off += round_up(mv, 256);
    plan->idx = off; off += round_up(mi, 256);
    plan->ws = off; off += round_up(ms, 256);
    plan->slot = off;
    plan->total = 2 * off;
    return true;
}
}  // namespace

size_t elsa_vit_host_device_bytes(const elsa_host_layer* cfg, int n_layers, elsa_dtype dtype)
{
    HostPlan plan;
    if (!cfg || n_layers <= 0 || !host_plan(cfg, n_layers, dtype, &plan)) return 0;
    return plan.total;
}

elsa_status elsa_vit_linears_host(const elsa_host_layer* cfg, int n_layers, elsa_dtype dtype, void* device_mem,
                                  size_t device_bytes, uint32_t* dev_status, void* stream_)
{
    if (!cfg) return fail(ELSA_ERR_NULL, "cfg must not be NULL");
    if (n_layers <= 0) return fail(ELSA_ERR_SHAPE, "non-positive n_layers=%d", n_layers);
    HostPlan plan;
    if (!host_plan(cfg, n_layers, dtype, &plan)) return fail(ELSA_ERR_SHAPE, "a layer has a non-positive dimension");
    for (int l = 0; l < n_layers; ++l) {
        const elsa_host_layer& c = cfg[l];
        if (!c.X || !c.Y || !c.W) return fail(ELSA_ERR_NULL, "layer %d: X, Y and W must not be NULL", l);
        elsa_status st = check_level(c.out, c.in, c.N, c.M, dtype);
        if (st != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "layer %d: %s", l, msg);
        }
    }
    if (!device_mem || device_bytes < plan.total)
        return fail(ELSA_ERR_WORKSPACE, "device memory of %zu bytes needed, %zu given", plan.total,
                    device_mem ? device_bytes : (size_t)0);
    if (((uintptr_t)device_mem & 255u) != 0) return fail(ELSA_ERR_ALIGN, "device_mem must be 256-byte aligned");
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;

    cudaStream_t stream = (cudaStream_t)stream_;
    HostPipe* pipe = nullptr;
    if ((st = host_pipe(dev.device, &pipe)) != ELSA_OK) return st;
    // Three queues: host-to-device copies, kernels (the caller's stream), device-to-host copies.  Layer l
    // uses slot l % 2; events order a slot's copy-in after the kernels that last read it, its kernels after
    // its copy-in and after the copy-out that last read its Y, and its copy-out after its kernels.
    auto cuda_fail = [](cudaError_t e, int l, const char* what) {
        cudaGetLastError();
        set_profile_layer(-1);
        return fail(ELSA_ERR_CUDA, "layer %d: %s: %s", l, what, cudaGetErrorString(e));
    };
    cudaError_t e = cudaEventRecord(pipe->start, stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->in, pipe->start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->out, pipe->start, 0);
    if (e != cudaSuccess) return cuda_fail(e, 0, "ordering the copy streams");
    for (int l = 0; l < n_layers; ++l) {
        const elsa_host_layer& c = cfg[l];
        const int slot = l & 1;
        uint8_t* base = (uint8_t*)device_mem + (size_t)slot * plan.slot;
        set_profile_layer(l);
        void* dX = base + plan.x; void* dY = base + plan.y; void* dW = base + plan.w;
        void* dB = c.bias ? base + plan.bias : nullptr;
        void* dV = base + plan.vals; uint32_t* dI = c.N == c.M ? nullptr : (uint32_t*)(base + plan.idx);
        // copy-in
        e = cudaSuccess;
        if (l >= 2) e = cudaStreamWaitEvent(pipe->in, pipe->compute_done[slot], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dW, c.W, (size_t)c.out * c.in * 2, cudaMemcpyHostToDevice, pipe->in);
        if (e == cudaSuccess && c.bias) e = cudaMemcpyAsync(dB, c.bias, (size_t)c.out * 2, cudaMemcpyHostToDevice, pipe->in);
        if (e == cudaSuccess) e = cudaMemcpyAsync(dX, c.X, (size_t)c.rows * c.in * 2, cudaMemcpyHostToDevice, pipe->in);
        if (e == cudaSuccess) e = cudaEventRecord(pipe->in_done[slot], pipe->in);
        if (e != cudaSuccess) return cuda_fail(e, l, "host-to-device copy");
        // kernels
        e = cudaStreamWaitEvent(stream, pipe->in_done[slot], 0);
        if (e == cudaSuccess && l >= 2) e = cudaStreamWaitEvent(stream, pipe->out_done[slot], 0);
        if (e != cudaSuccess) return cuda_fail(e, l, "ordering the kernels");
        if ((st = launch_compress((const uint16_t*)dW, c.out, c.in, c.N, c.M, (uint16_t*)dV, dI, stream)) != ELSA_OK) return st;
        if ((st = run_linear(dX, c.rows, dV, dI, dB, c.out, c.in, c.N, c.M, dtype, dY, base + plan.ws, dev_status,
                             stream)) != ELSA_OK)
            return st;
        e = cudaEventRecord(pipe->compute_done[slot], stream);
        // copy-out
        if (e == cudaSuccess) e = cudaStreamWaitEvent(pipe->out, pipe->compute_done[slot], 0);
        if (e == cudaSuccess) e = cudaMemcpyAsync(c.Y, dY, (size_t)c.rows * c.out * 2, cudaMemcpyDeviceToHost, pipe->out);
        if (e == cudaSuccess) e = cudaEventRecord(pipe->out_done[slot], pipe->out);
        if (e != cudaSuccess) return cuda_fail(e, l, "device-to-host copy");
    }
    set_profile_layer(-1);
    // the caller's stream is complete only when the last copies out are
    e = cudaStreamWaitEvent(stream, pipe->out_done[(n_layers - 1) & 1], 0);
    if (e == cudaSuccess && n_layers >= 2) e = cudaStreamWaitEvent(stream, pipe->out_done[n_layers & 1], 0);
    if (e != cudaSuccess) return cuda_fail(e, n_layers - 1, "joining the copy streams");
    return ELSA_OK;
}

}  // extern "C"

/* ---------------------------------------------------------------------------------------------- */
/* The chained block                                                                              */
/* ---------------------------------------------------------------------------------------------- */
namespace elsa {
namespace {

struct BlockLinear {
    const elsa_block_linear* w;
    int in, out;
    LinearKind kind;
    void* ws;          // this linear's part of region WORKSPACE
    bool image_ready;  // its weight image has been enqueued already
};

struct BlockPlan {
    size_t off[ELSA_BLOCK_REGIONS];
    size_t ws_off[4];   // qkv, proj, fc1, fc2 inside region WORKSPACE
    size_t total;
};

bool block_plan(int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype, BlockPlan* p)
{
    if (!w || rows <= 0 || dim <= 0 || mlp_dim <= 0 || dim % 8 != 0 || mlp_dim % 8 != 0) return false;
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return false;
    const size_t row = (size_t)rows * 2;
    const size_t sizes[7] = {row * dim, row * dim * 3, row * dim, row * dim, row * dim, row * mlp_dim, row * dim};
    size_t at = 0;
    for (int r = 0; r < 7; ++r) {
        p->off[r] = at;
        at += round_up(sizes[r], 256);
    }
    p->off[ELSA_BLOCK_WORKSPACE] = at;
    const elsa_block_linear* lin[4] = {&w->qkv, &w->proj, &w->fc1, &w->fc2};
    const int ins[4] = {dim, dim, dim, mlp_dim}, outs[4] = {3 * dim, dim, mlp_dim, dim};
    for (int l = 0; l < 4; ++l) {
        if (index_bits(lin[l]->M) < 0 || lin[l]->N < 1 || lin[l]->N > lin[l]->M || ins[l] % lin[l]->M != 0) return false;
        p->ws_off[l] = at;
        at += round_up(elsa_workspace_bytes(rows, ins[l], outs[l], lin[l]->N, lin[l]->M, dtype), 256);
    }
    p->total = at;
    return true;
}

// Validation shared by the three entry points; fills the four linears' descriptions.
elsa_status block_check(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                        const void* y, bool need_y, void* scratch, size_t scratch_bytes, BlockPlan* plan,
                        BlockLinear (&lin)[4], const DeviceInfo& dev)
{
    if (!x || !w || !scratch || (need_y && !y)) return fail(ELSA_ERR_NULL, "x, w, y and scratch must not be NULL");
    if (rows <= 0 || dim <= 0 || mlp_dim <= 0) return fail(ELSA_ERR_SHAPE, "non-positive size (rows=%d, dim=%d, mlp_dim=%d)", rows, dim, mlp_dim);
    if (!w->ln1_gain || !w->ln1_bias || !w->ln2_gain || !w->ln2_bias)
        return fail(ELSA_ERR_NULL, "the LayerNorm gains and biases must not be NULL");
    if (!(w->eps >= 0.f)) return fail(ELSA_ERR_SHAPE, "eps must not be negative");
    const elsa_block_linear* src[4] = {&w->qkv, &w->proj, &w->fc1, &w->fc2};
    const char* names[4] = {"qkv", "proj", "fc1", "fc2"};
    const int ins[4] = {dim, dim, dim, mlp_dim}, outs[4] = {3 * dim, dim, mlp_dim, dim};
    for (int l = 0; l < 4; ++l) {
        elsa_status st = check_level(outs[l], ins[l], src[l]->N, src[l]->M, dtype);
        if (st == ELSA_OK && !src[l]->vals) st = fail(ELSA_ERR_NULL, "vals must not be NULL");
        if (st == ELSA_OK && src[l]->N != src[l]->M && !src[l]->idx) st = fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
        if (st == ELSA_OK && (!aligned16(src[l]->vals) || (src[l]->idx && !aligned16(src[l]->idx)) ||
                              (src[l]->bias && !aligned16(src[l]->bias))))
            st = fail(ELSA_ERR_ALIGN, "vals, idx and bias must be 16-byte aligned");
        if (st != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "%s: %s", names[l], msg);
        }
    }
    if (!aligned16(x) || (y && !aligned16(y)) || !aligned16(w->ln1_gain) || !aligned16(w->ln1_bias) ||
        !aligned16(w->ln2_gain) || !aligned16(w->ln2_bias))
        return fail(ELSA_ERR_ALIGN, "x, y and the LayerNorm parameters must be 16-byte aligned");
    if (y && y == x) return fail(ELSA_ERR_ALIGN, "y may not alias x");
    if (!block_plan(rows, dim, mlp_dim, w, dtype, plan)) return fail(ELSA_ERR_SHAPE, "dim and mlp_dim must be multiples of 8");
    if (((uintptr_t)scratch & 255u) != 0) return fail(ELSA_ERR_ALIGN, "scratch must be 256-byte aligned");
    if (scratch_bytes < plan->total)
        return fail(ELSA_ERR_WORKSPACE, "scratch of %zu bytes needed, %zu given", plan->total, scratch_bytes);
    for (int l = 0; l < 4; ++l) {
        lin[l].w = src[l];
        lin[l].in = ins[l];
        lin[l].out = outs[l];
        lin[l].ws = (uint8_t*)scratch + plan->ws_off[l];
        lin[l].image_ready = false;
        elsa_status st = pick_kind(rows, outs[l], ins[l], src[l]->N, src[l]->M, dev.sm_count, &lin[l].kind);
        if (st != ELSA_OK) return st;
    }
    return ELSA_OK;
}

// The weight image of a linear whose kernel takes it ready-made (the others build theirs when they run).
elsa_status block_image(BlockLinear& L, cudaStream_t stream)
{
    const elsa_block_linear& w = *L.w;
    elsa_status st = ELSA_OK;
    if (w.N == w.M) return ELSA_OK;
    if (L.kind == KIND_DENSE_PAIR)
        st = launch_unpack((const uint16_t*)w.vals, w.idx, L.out, L.in, w.N, w.M, (uint16_t*)L.ws, stream);
    else if (L.kind == KIND_SPARSE_WS)
        st = launch_linear_tc_sparse_pair_prepare((const uint16_t*)w.vals, w.idx, L.out, L.in, w.N, w.M, SP24_PERMUTED,
                                                  L.ws, stream);
    else if (L.kind == KIND_SPARSE_ST)
        st = launch_nm_to_sp24((const uint16_t*)w.vals, w.idx, L.out, L.in, w.N, w.M, 128, SP24_TILED, (uint16_t*)L.ws,
                               (uint8_t*)L.ws + sp24_meta_offset(L.out, L.in), stream);
    else
        return ELSA_OK;
    L.image_ready = st == ELSA_OK;
    return st;
}

// Y = act(X Wm^T + bias) [+ residual].  Returns in *residual_left whether the residual is still to be added:
// then the linear's output went to `tmp` instead of Y, rounded to 16 bits.
elsa_status block_linear(BlockLinear& L, const uint16_t* X, int rows, elsa_dtype dtype, uint16_t* Y, int act,
                         const uint16_t* residual, uint16_t* tmp, bool* residual_left, uint32_t* dev_status,
                         cudaStream_t stream)
{
    const elsa_block_linear& w = *L.w;
    elsa_status st = ELSA_OK;
    *residual_left = false;
    if (L.kind == KIND_DENSE_PAIR) {
        if (w.N != w.M && !L.image_ready && (st = block_image(L, stream)) != ELSA_OK) return st;
        PairJob job;
        job.X = X; job.Wd = w.N == w.M ? (const uint16_t*)w.vals : (const uint16_t*)L.ws;
        job.bias = (const uint16_t*)w.bias; job.Y = Y;
        job.rows = rows; job.in = L.in; job.out = L.out;
        job.act = act; job.residual = residual;
        return launch_linear_tc_pair_group(&job, 1, dtype, dev_status, stream);
    }
    *residual_left = residual != nullptr;
    uint16_t* dst = residual ? tmp : Y;
    if (L.kind == KIND_SPARSE_WS || L.kind == KIND_SPARSE_ST) {
        if (!L.image_ready && (st = block_image(L, stream)) != ELSA_OK) return st;
        SparseJob job;
        job.X = X; job.bias = (const uint16_t*)w.bias; job.Y = dst; job.workspace = L.ws;
        job.rows = rows; job.in = L.in; job.out = L.out; job.act = act;
        return L.kind == KIND_SPARSE_WS ? launch_linear_tc_sparse_ws_group(&job, 1, dtype, dev_status, stream)
                                        : launch_linear_tc_sparse_st_group(&job, 1, dtype, dev_status, stream);
    }
    st = run_linear(X, rows, w.vals, w.N == w.M ? nullptr : w.idx, w.bias, L.out, L.in, w.N, w.M, dtype, dst, L.ws,
                    dev_status, stream);
    if (st != ELSA_OK) return st;
    return launch_act_inplace(dst, (long long)rows * L.out, act, dtype, stream);
}

// What a block leaves to its successor when the residual of its last linear has not been added yet: the block's
// output is t + r, and the successor's first LayerNorm adds, stores and normalises it in one pass.
struct BlockCarry {
    const uint16_t* t = nullptr;   // fc2's output, rounded to 16 bits
    const uint16_t* r = nullptr;   // x2
};

// carry (or NULL) + x_sum: the block's input is carry->t + carry->r, written to x_sum; otherwise it is x.
elsa_status block_qkv(const uint16_t* x, int rows, int dim, const elsa_block_weights* w, elsa_dtype dtype,
                      uint8_t* scratch, const BlockPlan& plan, BlockLinear (&lin)[4], uint32_t* dev_status,
                      cudaStream_t stream, const BlockCarry* carry = nullptr, uint16_t* x_sum = nullptr,
                      const elsa_swin_attn* swin = nullptr)
{
    uint16_t* x1 = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_X1]);
    uint16_t* qkv = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_QKV]);
    const bool add = carry != nullptr && carry->t != nullptr;
    RowMap out_map = {0, 0, 0, 0, 0, 1};      // Swin: x1 is written in window order, so that windows are runs of rows
    if (swin) { out_map.H = swin->H; out_map.W = swin->W; out_map.ws = swin->window; out_map.shift = swin->shift; }
    elsa_status st = launch_layer_norm(add ? carry->t : x, add ? carry->r : nullptr, add ? x_sum : nullptr,
                                       (const uint16_t*)w->ln1_gain, (const uint16_t*)w->ln1_bias,
                                       x1, rows, dim, w->eps, dtype, stream, swin ? &out_map : nullptr);
    if (st != ELSA_OK) return st;
    bool left = false;
    return block_linear(lin[0], x1, rows, dtype, qkv, 0, nullptr, nullptr, &left, dev_status, stream);
}

elsa_status block_rest(const uint16_t* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                       uint16_t* y, uint8_t* scratch, const BlockPlan& plan, BlockLinear (&lin)[4],
                       uint32_t* dev_status, cudaStream_t stream, BlockCarry* defer = nullptr,
                       const elsa_swin_attn* swin = nullptr)
{
    (void)mlp_dim;
    const uint16_t* a = (const uint16_t*)(scratch + plan.off[ELSA_BLOCK_A]);
    uint16_t* x2 = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_X2]);
    uint16_t* x3 = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_X3]);
    uint16_t* h = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_H]);
    uint16_t* t = (uint16_t*)(scratch + plan.off[ELSA_BLOCK_T]);
    const uint16_t* g2 = (const uint16_t*)w->ln2_gain;
    const uint16_t* b2 = (const uint16_t*)w->ln2_bias;
    bool left = false;
    elsa_status st;
    if (swin) {
        // proj runs on rows in window order; the add that follows reads them back in the grid's order
        RowMap in_map = {swin->H, swin->W, swin->window, swin->shift, 1, 0};
        if ((st = block_linear(lin[1], a, rows, dtype, t, 0, nullptr, nullptr, &left, dev_status, stream)) != ELSA_OK) return st;
        st = launch_layer_norm(t, x, x2, g2, b2, x3, rows, dim, w->eps, dtype, stream, &in_map);
    } else {
        if ((st = block_linear(lin[1], a, rows, dtype, x2, 0, x, t, &left, dev_status, stream)) != ELSA_OK) return st;
        // x2 = x + proj(a) and x3 = LayerNorm2(x2): one pass where the residual is still to be added
        st = left ? launch_layer_norm(t, x, x2, g2, b2, x3, rows, dim, w->eps, dtype, stream)
                  : launch_layer_norm(x2, nullptr, nullptr, g2, b2, x3, rows, dim, w->eps, dtype, stream);
    }
    if (st != ELSA_OK) return st;
    if ((st = block_linear(lin[2], x3, rows, dtype, h, 1, nullptr, nullptr, &left, dev_status, stream)) != ELSA_OK) return st;
    if ((st = block_linear(lin[3], h, rows, dtype, y, 0, x2, t, &left, dev_status, stream)) != ELSA_OK) return st;
    if (left && defer != nullptr) {          // the successor's first LayerNorm adds the residual
        defer->t = t;
        defer->r = x2;
        return ELSA_OK;
    }
    if (left) st = launch_layer_norm(t, x2, y, nullptr, nullptr, nullptr, rows, dim, w->eps, dtype, stream);
    return st;
}

}  // namespace
}  // namespace elsa

extern "C" {

size_t elsa_vit_block_scratch_bytes(int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                                    size_t* offsets)
{
    BlockPlan plan;
    if (!block_plan(rows, dim, mlp_dim, w, dtype, &plan)) return 0;
    if (offsets)
        for (int r = 0; r < ELSA_BLOCK_REGIONS; ++r) offsets[r] = plan.off[r];
    return plan.total;
}

elsa_status elsa_vit_block_qkv(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w,
                               elsa_dtype dtype, void* scratch, size_t scratch_bytes, uint32_t* dev_status, void* stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    BlockPlan plan;
    BlockLinear lin[4];
    if ((st = block_check(x, rows, dim, mlp_dim, w, dtype, nullptr, false, scratch, scratch_bytes, &plan, lin, dev)) != ELSA_OK)
        return st;
    return block_qkv((const uint16_t*)x, rows, dim, w, dtype, (uint8_t*)scratch, plan, lin, dev_status, (cudaStream_t)stream);
}

elsa_status elsa_vit_block_rest(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w,
                                elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes, uint32_t* dev_status,
                                void* stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    BlockPlan plan;
    BlockLinear lin[4];
    if ((st = block_check(x, rows, dim, mlp_dim, w, dtype, y, true, scratch, scratch_bytes, &plan, lin, dev)) != ELSA_OK)
        return st;
    return block_rest((const uint16_t*)x, rows, dim, mlp_dim, w, dtype, (uint16_t*)y, (uint8_t*)scratch, plan, lin,
                      dev_status, (cudaStream_t)stream);
}

}  // extern "C"

namespace elsa {
namespace {

// The whole block; tokens == 0 runs the stand-in a = V, otherwise the attention kernel over images of `tokens` rows.
elsa_status run_block(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                      void* y, void* scratch, size_t scratch_bytes, uint32_t* dev_status, void* stream_, int tokens, int heads,
                      const BlockCarry* carry = nullptr, uint16_t* x_sum = nullptr, BlockCarry* defer = nullptr,
                      const elsa_swin_attn* swin = nullptr)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    BlockPlan plan;
    BlockLinear lin[4];
    if ((st = block_check(x, rows, dim, mlp_dim, w, dtype, y, true, scratch, scratch_bytes, &plan, lin, dev)) != ELSA_OK)
        return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    // The four weight images do not depend on x: they are built on the library's side stream while the first
    // LayerNorm runs on the caller's, which waits for them before the first linear.
    bool any_image = false;
    for (int l = 0; l < 4; ++l)
        any_image = any_image || (lin[l].w->N != lin[l].w->M && (lin[l].kind == KIND_DENSE_PAIR ||
                                                                  lin[l].kind == KIND_SPARSE_WS || lin[l].kind == KIND_SPARSE_ST));
    SidePipe* side = nullptr;
    if (any_image) {
        if ((st = side_pipe(dev.device, &side)) != ELSA_OK) return st;
        cudaError_t e = cudaEventRecord(side->fork, stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(side->stream, side->fork, 0);
        if (e != cudaSuccess) return fail(ELSA_ERR_CUDA, "forking the image stream: %s", cudaGetErrorString(e));
        for (int l = 0; l < 4 && st == ELSA_OK; ++l) st = block_image(lin[l], side->stream);
        e = cudaEventRecord(side->join, side->stream);   // joined even after a failed launch: the fork must not dangle
        if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, side->join, 0);
        if (st != ELSA_OK) return st;
        if (e != cudaSuccess) return fail(ELSA_ERR_CUDA, "joining the image stream: %s", cudaGetErrorString(e));
    }
    uint8_t* s8 = (uint8_t*)scratch;
    if ((st = block_qkv((const uint16_t*)x, rows, dim, w, dtype, s8, plan, lin, dev_status, stream, carry, x_sum, swin)) != ELSA_OK)
        return st;
    if (carry != nullptr && carry->t != nullptr) x = x_sum;      // the block's input, as just stored
    if (swin) {
        const int pack = swin->pack < 1 ? 1 : swin->pack;
        const int T = swin->window * swin->window * pack;
        st = launch_attention((const uint16_t*)(s8 + plan.off[ELSA_BLOCK_QKV]), rows / T, T, heads, dim, dtype,
                              (uint16_t*)(s8 + plan.off[ELSA_BLOCK_A]), dev_status, stream, swin->rel_bias,
                              swin->shift > 0 ? swin->mask : nullptr, (swin->H / swin->window) * (swin->W / swin->window) / pack,
                              swin->bias_pitch);
    } else if (tokens == 0) {
        // the stated stand-in for attention: a = V
        st = launch_copy_columns((const uint16_t*)(s8 + plan.off[ELSA_BLOCK_QKV]), (uint16_t*)(s8 + plan.off[ELSA_BLOCK_A]),
                                 rows, 3 * dim, 2 * dim, dim, stream);
    } else {
        st = launch_attention((const uint16_t*)(s8 + plan.off[ELSA_BLOCK_QKV]), rows / tokens, tokens, heads, dim, dtype,
                              (uint16_t*)(s8 + plan.off[ELSA_BLOCK_A]), dev_status, stream);
    }
    if (st != ELSA_OK) return st;
    return block_rest((const uint16_t*)x, rows, dim, mlp_dim, w, dtype, (uint16_t*)y, s8, plan, lin, dev_status, stream, defer, swin);
}

struct EncoderPlan {
    size_t block_bytes;   // scratch of the largest block
    size_t buf[2];        // byte offsets of the two activation buffers the blocks alternate between
    size_t total;
};

bool encoder_plan(int rows, int dim, int mlp_dim, const elsa_block_weights* blocks, int n_blocks, elsa_dtype dtype, EncoderPlan* p)
{
    if (!blocks || n_blocks <= 0) return false;
    p->block_bytes = 0;
    for (int b = 0; b < n_blocks; ++b) {
        BlockPlan plan;
        if (!block_plan(rows, dim, mlp_dim, blocks + b, dtype, &plan)) return false;
        if (plan.total > p->block_bytes) p->block_bytes = plan.total;
    }
    size_t at = round_up(p->block_bytes, 256);
    for (int i = 0; i < 2; ++i) {
        p->buf[i] = at;
        at += round_up((size_t)rows * dim * 2, 256);
    }
    p->total = at;
    return true;
}

}  // namespace
}  // namespace elsa

extern "C" {

size_t elsa_vit_encoder_scratch_bytes(int images, int tokens, int dim, int mlp_dim, const elsa_block_weights* blocks,
                                      int n_blocks, elsa_dtype dtype)
{
    EncoderPlan p;
    if (images <= 0 || tokens <= 0 || (long long)images * tokens > 0x7fffffffLL) return 0;
    return encoder_plan(images * tokens, dim, mlp_dim, blocks, n_blocks, dtype, &p) ? p.total : 0;
}

elsa_status elsa_vit_encoder(const void* x, int images, int tokens, int heads, int dim, int mlp_dim,
                             const elsa_block_weights* blocks, int n_blocks, const void* final_gain, const void* final_bias,
                             float final_eps, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                             uint32_t* dev_status, void* stream)
{
    if (!x || !y || !blocks || !scratch) return fail(ELSA_ERR_NULL, "x, y, blocks and scratch must not be NULL");
    if (images <= 0 || tokens <= 0 || n_blocks <= 0)
        return fail(ELSA_ERR_SHAPE, "non-positive images=%d, tokens=%d or n_blocks=%d", images, tokens, n_blocks);
    if (!attention_suits(tokens, heads, dim))
        return fail(ELSA_ERR_SHAPE, "attention needs at most 256 tokens per image and dim = 64 * heads (tokens=%d, heads=%d, dim=%d)",
                    tokens, heads, dim);
    if ((long long)images * tokens > 0x7fffffffLL) return fail(ELSA_ERR_SHAPE, "images * tokens does not fit an int");
    if ((final_gain == nullptr) != (final_bias == nullptr)) return fail(ELSA_ERR_NULL, "final_gain and final_bias go together");
    if (final_gain && (!aligned16(final_gain) || !aligned16(final_bias)))
        return fail(ELSA_ERR_ALIGN, "final_gain and final_bias must be 16-byte aligned");
    if (final_gain && !(final_eps >= 0.f)) return fail(ELSA_ERR_SHAPE, "final_eps must not be negative");
    const int rows = images * tokens;
    EncoderPlan plan;
    if (!encoder_plan(rows, dim, mlp_dim, blocks, n_blocks, dtype, &plan))
        return fail(ELSA_ERR_SHAPE, "dim and mlp_dim must be multiples of 8 and every level valid");
    if (((uintptr_t)scratch & 255u) != 0) return fail(ELSA_ERR_ALIGN, "scratch must be 256-byte aligned");
    if (scratch_bytes < plan.total) return fail(ELSA_ERR_WORKSPACE, "scratch of %zu bytes needed, %zu given", plan.total, scratch_bytes);
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    uint8_t* s8 = (uint8_t*)scratch;
    uint16_t* buf[2] = {(uint16_t*)(s8 + plan.buf[0]), (uint16_t*)(s8 + plan.buf[1])};
    // every block is validated before the first launch
    for (int b = 0; b < n_blocks; ++b) {
        BlockPlan bp;
        BlockLinear lin[4];
        if ((st = block_check(x, rows, dim, mlp_dim, blocks + b, dtype, buf[0], true, scratch, plan.block_bytes, &bp, lin, dev)) != ELSA_OK) {
            char msg[400];
            snprintf(msg, sizeof msg, "%s", elsa_last_error());
            return fail(st, "block %d: %s", b, msg);
        }
    }
    // Block b reads its input from buf[b % 2] (block 0: from x) and writes its output to buf[(b + 1) % 2]; where a
    // block's last residual is still to be added, the next block's first LayerNorm does it while it normalises.
    BlockCarry carry;
    const void* in = x;
    for (int b = 0; b < n_blocks; ++b) {
        const bool last = b + 1 == n_blocks;
        void* out = (last && final_gain == nullptr) ? y : (void*)buf[(b + 1) & 1];
        BlockCarry next;
        st = run_block(in, rows, dim, mlp_dim, blocks + b, dtype, out, scratch, plan.block_bytes, dev_status, stream, tokens, heads,
                       &carry, buf[b & 1], last && final_gain == nullptr ? nullptr : &next);
        if (st != ELSA_OK) return st;
        carry = next;
        in = buf[(b + 1) & 1];
    }
    if (final_gain != nullptr) {
        const bool add = carry.t != nullptr;
        st = launch_layer_norm(add ? carry.t : buf[n_blocks & 1], add ? carry.r : nullptr, add ? buf[n_blocks & 1] : nullptr,
                               (const uint16_t*)final_gain, (const uint16_t*)final_bias, (uint16_t*)y, rows, dim, final_eps, dtype,
                               (cudaStream_t)stream);
    }
    return st;
}

elsa_status elsa_vit_block(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                           void* y, void* scratch, size_t scratch_bytes, uint32_t* dev_status, void* stream)
{
    return run_block(x, rows, dim, mlp_dim, w, dtype, y, scratch, scratch_bytes, dev_status, stream, 0, 0);
}

elsa_status elsa_attention(const void* qkv, int images, int tokens, int heads, int dim, elsa_dtype dtype, void* a,
                           uint32_t* dev_status, void* stream)
{
    if (!qkv || !a) return fail(ELSA_ERR_NULL, "qkv and a must not be NULL");
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return fail(ELSA_ERR_DTYPE, "dtype %d is neither ELSA_F16 nor ELSA_BF16", (int)dtype);
    if (images <= 0) return fail(ELSA_ERR_SHAPE, "non-positive images=%d", images);
    if (!aligned16(qkv) || !aligned16(a)) return fail(ELSA_ERR_ALIGN, "qkv and a must be 16-byte aligned");
    return launch_attention((const uint16_t*)qkv, images, tokens, heads, dim, dtype, (uint16_t*)a, dev_status, (cudaStream_t)stream);
}

int elsa_swin_mask(int H, int W, int window, int shift, int pack, int pitch, float* mask)
{
    if (H <= 0 || W <= 0 || window <= 0 || H % window != 0 || W % window != 0 || shift <= 0 || shift >= window || pack < 1 ||
        pitch < pack * window * window || !mask)
        return -1;
    const int T = window * window, nww = W / window, n_windows = (H / window) * nww;
    if (n_windows % pack != 0) return -1;
    // region of a position of the rolled grid: the bands [0, n - window), [n - window, n - shift), [n - shift, n) of each axis
    auto band = [&](int v, int n) { return v < n - window ? 0 : v < n - shift ? 1 : 2; };
    auto region = [&](int win, int t) {
        const int wi = win / nww, wj = win % nww;
        return 3 * band(wi * window + t / window, H) + band(wj * window + t % window, W);
    };
    for (int g = 0; g < n_windows / pack; ++g) {
        float* m = mask + (size_t)g * pack * T * pitch;
        for (int p = 0; p < pack * T; ++p)
            for (int q = 0; q < pitch; ++q) {
                float v = 0.f;
                // tokens of different windows of a group are kept apart by the bias table; here: the seam inside a window
                if (q < pack * T && p / T == q / T) v = region(g * pack + p / T, p % T) != region(g * pack + q / T, q % T) ? -100.f : 0.f;
                m[(size_t)p * pitch + q] = v;
            }
    }
    return n_windows / pack;
}

int elsa_swin_pack_bias(const float* rel_bias, int heads, int window, int pack, int pitch, float* packed)
{
    if (!rel_bias || !packed || heads <= 0 || window <= 0 || pack < 1 || pitch < pack * window * window) return -1;
    const int T = window * window;
    for (int h = 0; h < heads; ++h)
        for (int p = 0; p < pack * T; ++p)
            for (int q = 0; q < pitch; ++q) {
                float v = 0.f;
                if (q < pack * T) v = p / T == q / T ? rel_bias[((size_t)h * T + p % T) * T + q % T] : -30000.f;
                packed[((size_t)h * pack * T + p) * pitch + q] = v;
            }
    return 0;
}

elsa_status elsa_swin_block(const void* x, int images, int heads, int dim, int mlp_dim, const elsa_block_weights* w,
                            const elsa_swin_attn* attn, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                            uint32_t* dev_status, void* stream)
{
    if (!attn) return fail(ELSA_ERR_NULL, "attn must not be NULL");
    if (images <= 0 || attn->H <= 0 || attn->W <= 0 || attn->window <= 0 || attn->H % attn->window != 0 ||
        attn->W % attn->window != 0 || attn->shift < 0 || attn->shift >= attn->window)
        return fail(ELSA_ERR_SHAPE, "windows of %d do not tile a %d x %d grid, or shift=%d is outside [0, window)", attn->window,
                    attn->H, attn->W, attn->shift);
    const int pack = attn->pack < 1 ? 1 : attn->pack;
    const int T = attn->window * attn->window * pack;         // tokens of one attention item: `pack` windows
    if (!attention_suits(T, heads, dim))
        return fail(ELSA_ERR_SHAPE, "window attention needs at most 256 tokens per group of windows and dim = 32 or 64 times heads "
                    "(window=%d, pack=%d, heads=%d, dim=%d)", attn->window, pack, heads, dim);
    if (((long long)images * (attn->H / attn->window) * (attn->W / attn->window)) % pack != 0)
        return fail(ELSA_ERR_SHAPE, "the windows do not divide into groups of %d", pack);
    if (attn->shift > 0 && ((attn->H / attn->window) * (attn->W / attn->window)) % pack != 0)
        return fail(ELSA_ERR_SHAPE, "with a shift the windows of one image must divide into groups of %d", pack);
    if (!attn->rel_bias || (attn->shift > 0 && !attn->mask)) return fail(ELSA_ERR_NULL, "rel_bias (and mask when shift > 0) must not be NULL");
    if (attn->bias_pitch < T) return fail(ELSA_ERR_SHAPE, "bias_pitch=%d is below the %d tokens of a window", attn->bias_pitch, T);
    if ((long long)images * attn->H * attn->W > 0x7fffffffLL) return fail(ELSA_ERR_SHAPE, "images * H * W does not fit an int");
    return run_block(x, images * attn->H * attn->W, dim, mlp_dim, w, dtype, y, scratch, scratch_bytes, dev_status, stream, T, heads,
                     nullptr, nullptr, nullptr, attn);
}

elsa_status elsa_window_attention(const void* qkv, int windows, int tokens, int heads, int dim, const float* bias,
                                  int bias_pitch, const float* mask, int n_masks, elsa_dtype dtype, void* a,
                                  uint32_t* dev_status, void* stream)
{
    if (!qkv || !a || !bias) return fail(ELSA_ERR_NULL, "qkv, a and bias must not be NULL");
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return fail(ELSA_ERR_DTYPE, "dtype %d is neither ELSA_F16 nor ELSA_BF16", (int)dtype);
    if (windows <= 0) return fail(ELSA_ERR_SHAPE, "non-positive windows=%d", windows);
    if (!aligned16(qkv) || !aligned16(a) || ((uintptr_t)bias & 3u) || ((uintptr_t)mask & 3u))
        return fail(ELSA_ERR_ALIGN, "qkv and a must be 16-byte aligned, the tables 4-byte aligned");
    return launch_attention((const uint16_t*)qkv, windows, tokens, heads, dim, dtype, (uint16_t*)a, dev_status, (cudaStream_t)stream,
                            bias, mask, n_masks, bias_pitch);
}

elsa_status elsa_vit_block_attn(const void* x, int images, int tokens, int heads, int dim, int mlp_dim,
                                const elsa_block_weights* w, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                                uint32_t* dev_status, void* stream)
{
    if (images <= 0 || tokens <= 0) return fail(ELSA_ERR_SHAPE, "non-positive images=%d or tokens=%d", images, tokens);
    if (!attention_suits(tokens, heads, dim))
        return fail(ELSA_ERR_SHAPE, "attention needs at most 256 tokens per image and dim = 64 * heads (tokens=%d, heads=%d, dim=%d)",
                    tokens, heads, dim);
    if ((long long)images * tokens > 0x7fffffffLL) return fail(ELSA_ERR_SHAPE, "images * tokens does not fit an int");
    return run_block(x, images * tokens, dim, mlp_dim, w, dtype, y, scratch, scratch_bytes, dev_status, stream, tokens, heads);
}

}  // extern "C"

/* ---------------------------------------------------------------------------------------------- */
/* Backward pass                                                                                  */
/* ---------------------------------------------------------------------------------------------- */
namespace elsa {
namespace {

struct BackwardPlan {
    size_t wm, wmt, partial, sums, total;   // byte offsets of the regions
};

// Upper bound, from host arithmetic alone, of the ranges the dW product may be cut into: what a device of 256 SMs
// would use.  The call clamps its choice to it.
int wgrad_splits_bound(int in, int out)
{
    const long long tiles = (long long)((out + 255) / 256) * ((in + 255) / 256);
    long long s = 128 / tiles;
    if (s > 8) s = 8;
    return s < 1 ? 1 : (int)s;
}

BackwardPlan backward_plan(int rows, int in, int out)
{
    BackwardPlan p;
    size_t at = 0;
    p.wm = at;      at += round_up((size_t)out * in * 2, 256);                      // masked weight [out][in]
    p.wmt = at;     at += round_up((size_t)out * in * 2, 256);                      // its transpose [in][out]
    p.partial = at; at += round_up((size_t)((rows + 511) / 512) * out * 4, 256);    // column sums of dY per 512 rows
    const int bound = wgrad_splits_bound(in, out);                                  // fp32 sums of dW per range of rows
    p.sums = at;    at += bound > 1 ? round_up((size_t)bound * out * in * 4, 256) : 0;
    p.total = at;
    return p;
}

// Y [m][n] = A [m][k] . B [n][k]^T on the dense tensor-core kernels (no bias).
elsa_status dense_product(const uint16_t* A, int m, const uint16_t* B, int n, int k, elsa_dtype dtype, uint16_t* Y,
                          uint32_t* dev_status, cudaStream_t stream, int sm_count)
{
    const int variant = g_variant.load(std::memory_order_relaxed);
    const bool pair = variant == ELSA_VARIANT_TC_PAIR || (variant != ELSA_VARIANT_TC_DENSE && linear_tc_pair_suits(m, n, sm_count));
    return pair ? launch_linear_tc_pair(A, m, B, nullptr, n, k, dtype, Y, dev_status, stream)
                : launch_linear_tc_dense(A, m, B, nullptr, n, k, dtype, Y, dev_status, stream);
}

}  // namespace
}  // namespace elsa

extern "C" {

size_t elsa_backward_workspace_bytes(int rows, int in, int out, int N, int M, elsa_dtype dtype)
{
    if (rows <= 0 || out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    if (dtype != ELSA_F16 && dtype != ELSA_BF16) return 0;
    return backward_plan(rows, in, out).total;
}

elsa_status elsa_nm_linear_backward(const void* dY, const void* X, int rows, const void* vals, const uint32_t* idx,
                                    int out, int in, int N, int M, elsa_dtype dtype, void* dX, void* dW, void* db,
                                    void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream_)
{
    if (!dY) return fail(ELSA_ERR_NULL, "dY must not be NULL");
    elsa_status st = check_level(out, in, N, M, dtype);
    if (st != ELSA_OK) return st;
    if (rows <= 0) return fail(ELSA_ERR_SHAPE, "non-positive rows=%d", rows);
    if (dX && !vals) return fail(ELSA_ERR_NULL, "vals must not be NULL when dX is wanted");
    if (dW && !X) return fail(ELSA_ERR_NULL, "X must not be NULL when dW is wanted");
    if ((dX || dW) && N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(dY) || (X && !aligned16(X)) || (vals && !aligned16(vals)) || (idx && !aligned16(idx)) ||
        (dX && !aligned16(dX)) || (dW && !aligned16(dW)) || (db && !aligned16(db)))
        return fail(ELSA_ERR_ALIGN, "dY, X, vals, idx, dX, dW and db must be 16-byte aligned");
    const BackwardPlan plan = backward_plan(rows, in, out);
    if (!workspace || workspace_bytes < plan.total)
        return fail(ELSA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", plan.total, workspace ? workspace_bytes : (size_t)0);
    if (((uintptr_t)workspace & 255u) != 0) return fail(ELSA_ERR_ALIGN, "workspace must be 256-byte aligned");
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;
    uint8_t* ws = (uint8_t*)workspace;
    const uint16_t* dy = (const uint16_t*)dY;
    if (dX) {
        // dX = dY Wm: the forward GEMM with the transposed masked weight, reduction over `out`
        uint16_t* wm = (uint16_t*)(ws + plan.wm);
        uint16_t* wmt = (uint16_t*)(ws + plan.wmt);
        const uint16_t* dense = (const uint16_t*)vals;
        if (N != M) {
            if ((st = launch_unpack((const uint16_t*)vals, idx, out, in, N, M, wm, stream)) != ELSA_OK) return st;
            dense = wm;
        }
        if ((st = launch_transpose16(dense, wmt, out, in, out, stream)) != ELSA_OK) return st;
        if ((st = dense_product(dy, rows, wmt, in, out, dtype, (uint16_t*)dX, dev_status, stream, dev.sm_count)) != ELSA_OK) return st;
    }
    if (db && (st = launch_colsum(dy, rows, out, (float*)(ws + plan.partial), (uint16_t*)db, dtype, stream)) != ELSA_OK) return st;
    if (dW) {
        // dW = dY^T X, reduction over the token rows: both operands are read as they are stored (reduction index
        // outermost), then the mask
        // when 256 x 256 tiles alone leave SM pairs idle, the rows are cut into ranges summed afterwards
        int splits = linear_tc_pair_tn_splits(out, in, rows, dev.sm_count);
        if (splits > wgrad_splits_bound(in, out)) splits = wgrad_splits_bound(in, out);
        float* sums = (float*)(ws + plan.sums);
        if ((st = launch_linear_tc_pair_tn(dy, (const uint16_t*)X, out, in, rows, dtype, (uint16_t*)dW, splits, sums, dev_status,
                                           stream)) != ELSA_OK)
            return st;
        st = splits > 1 ? launch_wgrad_finish(sums, splits, idx, out, in, N, M, dtype, (uint16_t*)dW, stream)
                        : launch_mask_apply((uint16_t*)dW, idx, out, in, N, M, stream);
        if (st != ELSA_OK) return st;
    }
    return ELSA_OK;
}

}  // extern "C"

extern "C" {

elsa_status elsa_set_linear_variant(elsa_variant v)
{
    if (v != ELSA_VARIANT_AUTO && v != ELSA_VARIANT_SIMT && v != ELSA_VARIANT_TC_DENSE && v != ELSA_VARIANT_TC_PAIR &&
        v != ELSA_VARIANT_TC_SPARSE && v != ELSA_VARIANT_TC_SPARSE_PAIR && v != ELSA_VARIANT_TC_SPARSE_WS &&
        v != ELSA_VARIANT_TC_SPARSE_ST)
        return fail(ELSA_ERR_SHAPE, "unknown variant %d", (int)v);
    g_variant.store((int)v, std::memory_order_relaxed);
    return ELSA_OK;
}

void elsa_set_grouping(int on) { g_grouping.store(on != 0, std::memory_order_relaxed); }

elsa_variant elsa_get_linear_variant(void) { return (elsa_variant)g_variant.load(std::memory_order_relaxed); }

elsa_status elsa_profile_start(void)
{
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    for (auto& r : g_profile) { cudaEventDestroy(r.start); cudaEventDestroy(r.stop); }
    g_profile.clear();
    g_profile_on.store(true, std::memory_order_relaxed);
    return ELSA_OK;
}

int elsa_profile_stop(elsa_kernel_time* records, int capacity)
{
    g_profile_on.store(false, std::memory_order_relaxed);
    std::lock_guard<std::mutex> lock(g_profile_mutex);
    const int n = (int)g_profile.size();
    for (int i = 0; i < n; ++i) {
        ProfileRecord& r = g_profile[i];
        float ms = -1.f;
        if (cudaEventSynchronize(r.stop) != cudaSuccess || cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) {
            cudaGetLastError();
            ms = -1.f;
        }
        if (records && i < capacity) {
            records[i].kernel = r.kernel;
            records[i].layer = r.layer;
            records[i].ms = ms;
        }
        cudaEventDestroy(r.start);
        cudaEventDestroy(r.stop);
    }
    g_profile.clear();
    return n;
}

unsigned long long elsa_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* elsa_last_error(void) { return g_error; }

}  // extern "C"
