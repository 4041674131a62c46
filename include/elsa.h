/*
 * elsa.h -- C ABI of the B200 (sm_100a) N:M sparse-linear library.
 *
 * The calls follow the problem statement of ELSA (arXiv 2409.09708): a ViT's
 * linear modules (qkv, proj, fc1, fc2; Sec. 3, L = 4B) each carry a sparsity
 * level N:M; the weight of a module is projected onto that level by keeping
 * the N largest-magnitude values of every group of M consecutive weights
 * (Sec. 3.1, Eq. 1), stored as the kept values plus one log2(M)-bit index each
 * (Sec. 1; Sec. 2, Fig. 2 top), and multiplied with dense activations so that
 * the result is the exact product with the pruned matrix (Sec. 2, Fig. 2
 * bottom).
 *
 * Conventions for every call unless stated otherwise
 *   - Tensor pointers are DEVICE pointers owned by the caller.  Matrices are
 *     row-major and contiguous.  W is [out][in] as in nn.Linear: Y = X W^T + b.
 *     Groups of M run along `in` (the reduction dimension), aligned at
 *     multiples of M.
 *   - 16-bit floats (fp16 or bf16, chosen by elsa_dtype) for X, W, values,
 *     bias and Y; accumulation in fp32; one round-to-nearest-even at the end.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Calls enqueue work and return; they never synchronise and never
 *     allocate or free device memory.
 *   - Arguments are validated on the host before anything is launched.  A bad
 *     argument returns a status; nothing aborts, throws or prints.
 *     elsa_last_error() gives a thread-local message for the last failure.
 *   - Pointers must be 16-byte aligned and `in`, `out` multiples of 8 (row
 *     pitches are then multiples of 16 bytes), else ELSA_ERR_ALIGN.
 *   - Supported levels: M in {4, 8, 16}, 1 <= N <= M, in % M == 0.
 *   - The library requires a compute-capability 10.x device (ELSA_ERR_ARCH).
 *
 * Packed format (what elsa_nm_compress writes and the other calls read)
 *   vals: [out][in/M*N] 16-bit, the kept values of each group in ascending
 *         in-group position, bit patterns unchanged.
 *   idx : [out][words_per_row] uint32.  The position (0..M-1) of kept value t
 *         of group g is the b = log2(M)-bit field at bit offset (g*N + t)*b of
 *         the row's bitstream, least-significant bit first inside
 *         little-endian words; rows start on a word boundary,
 *         words_per_row = ceil(in/M*N*b / 32); pad bits are zero.
 *         N == M stores no indices: idx may be NULL and vals equals W.
 */
#ifndef ELSA_H
#define ELSA_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    ELSA_OK = 0,
    ELSA_ERR_NULL = 1,      /* a required pointer is NULL */
    ELSA_ERR_SHAPE = 2,     /* non-positive dimension, or in % M != 0 */
    ELSA_ERR_NM = 3,        /* M not in {4, 8, 16}, N < 1 or N > M */
    ELSA_ERR_DTYPE = 4,
    ELSA_ERR_ALIGN = 5,     /* pointer not 16-byte aligned, or in/out not a multiple of 8 */
    ELSA_ERR_WORKSPACE = 6, /* workspace NULL or smaller than elsa_workspace_bytes() */
    ELSA_ERR_CUDA = 7,      /* a CUDA runtime/driver call failed; see elsa_last_error() */
    ELSA_ERR_TIMEOUT = 8,   /* reported through dev_status: a bounded device-side wait gave up */
    ELSA_ERR_ARCH = 9       /* current device is not compute capability 10.x */
} elsa_status;

typedef enum { ELSA_F16 = 0, ELSA_BF16 = 1 } elsa_dtype;

/* Which kernel elsa_nm_linear uses.  AUTO is the product path; the others exist so that
 * tests can force every variant over the same input and require agreement. */
typedef enum {
    ELSA_VARIANT_AUTO = 0,
    ELSA_VARIANT_SIMT = 1,    /* CUDA-core kernel reading the packed form directly (slow; checks) */
    ELSA_VARIANT_TC_DENSE = 2, /* expand to a dense tile image, tcgen05 dense MMA, one CTA per tile */
    ELSA_VARIANT_TC_PAIR = 3,  /* same, CTA pairs sharing a 256-row tile (tcgen05 cta_group::2) */
    ELSA_VARIANT_TC_SPARSE = 4, /* N <= 2 only: re-encode as 2-of-4 + metadata, tcgen05 sparse MMA */
    ELSA_VARIANT_TC_SPARSE_PAIR = 5, /* the same on CTA pairs (256 features x 224 rows per pair) */
    ELSA_VARIANT_TC_SPARSE_WS = 6, /* N <= 2, in % 128 == 0, in <= 1024: CTA pairs that keep their 256-feature
                                    * weight block and its metadata in tensor memory for a whole layer */
    ELSA_VARIANT_TC_SPARSE_ST = 7  /* N <= 2, in % 128 == 0, any length: the weight block streams through
                                    * tensor memory in K chunks of 256, shared memory carries activations only */
} elsa_variant;

/* Sizes of the packed form (host-only arithmetic; 0 on invalid arguments). */
size_t elsa_nm_values_bytes(int out, int in, int N, int M, elsa_dtype dtype);
size_t elsa_nm_index_bytes(int out, int in, int N, int M); /* 0 when N == M */

/* Bytes of device scratch elsa_nm_linear needs for this problem (host-only arithmetic). */
size_t elsa_workspace_bytes(int rows, int in, int out, int N, int M, elsa_dtype dtype);

/*
 * Sec. 3.1, Eq. 1 with magnitude saliency, then the compressed form of Sec. 1 / Sec. 2.
 * In every group of M consecutive weights of a row keep the N of largest |w|; |w| is compared
 * exactly on the 15 magnitude bits (so +0 == -0), and among equals the lowest position wins,
 * so exactly N positions are kept and the result is unique.
 *   W    in : [out][in] dense weight
 *   vals out: [out][in/M*N]
 *   idx  out: [out][words_per_row], may be NULL iff N == M
 */
elsa_status elsa_nm_compress(const void* W, int out, int in, int N, int M, elsa_dtype dtype,
                             void* vals, uint32_t* idx, void* stream);

/*
 * Inverse of the compressed form: W_masked [out][in] with +0.0 at pruned positions and the kept
 * values, bit for bit, at theirs (Sec. 2, Fig. 2: the indices give each value's original position).
 */
elsa_status elsa_nm_unpack(const void* vals, const uint32_t* idx, int out, int in, int N, int M,
                           elsa_dtype dtype, void* W_masked, void* stream);

/*
 * Sec. 2, Fig. 2 bottom: Y[rows][out] = X[rows][in] * W_masked^T + bias, computed from the packed
 * weight; only kept weights contribute.  fp32 accumulation, one rounding to the 16-bit output.
 *   bias       : [out] 16-bit, or NULL
 *   workspace  : device scratch of at least elsa_workspace_bytes(...) bytes, 256-byte aligned;
 *                its contents are overwritten; calls that share it must be stream-ordered
 *   dev_status : optional device word.  The caller zeroes it; if a bounded wait inside the
 *                kernel ever gives up, the kernel stores ELSA_ERR_TIMEOUT | (site << 8) there and
 *                all its threads return without trapping.  Read it after synchronising.
 */
elsa_status elsa_nm_linear(const void* X, int rows, const void* vals, const uint32_t* idx,
                           const void* bias, int out, int in, int N, int M, elsa_dtype dtype,
                           void* Y, void* workspace, size_t workspace_bytes,
                           uint32_t* dev_status, void* stream);

/* One weight of a table: dense W in, packed form out (as for elsa_nm_compress). */
typedef struct {
    const void* W;   /* [out][in] device */
    void* vals;      /* [out][in/M*N] device, written */
    uint32_t* idx;   /* index words, device, written; NULL iff N == M */
    int out, in, N, M;
} elsa_weight;

/*
 * elsa_nm_compress for every weight of a table, each to its own level (Sec. 3.1 applied under a
 * layer-wise configuration alpha, Sec. 3), in one kernel launch per 256 weights.  `w` is a HOST
 * array; results are bit-identical to per-weight calls.  The table is validated before anything is
 * launched; elsa_last_error() names the offending entry.
 */
elsa_status elsa_vit_compress(const elsa_weight* w, int n_weights, elsa_dtype dtype, void* stream);

/*
 * Sec. 3.1, subset-superset relation: all levels N:M of a supernet layer share one weight, and the
 * magnitude ranks inside a group do not depend on N.  This call reads W once and writes the packed
 * form of every requested level N_list[l]:M (same M), each bit-identical to what elsa_nm_compress
 * writes for that level.  `N_list`, `vals` and `idx` are HOST arrays of n_levels entries holding
 * device pointers (idx[l] may be NULL iff N_list[l] == M); n_levels <= 16.
 */
elsa_status elsa_nm_compress_levels(const void* W, int out, int in, int M, const int* N_list, int n_levels,
                                    elsa_dtype dtype, void* const* vals, uint32_t* const* idx, void* stream);

/*
 * Sec. 3.1 "dynamic masking" as the supernet's forward uses it (Alg. 2: the shared weight is
 * projected to the sampled level on every step): Y = X * (W_sup projected onto N:M)^T + bias
 * straight from the dense shared weight W_sup [out][in], with no packed copy.  The projection is
 * the one elsa_nm_compress defines, so the result equals elsa_nm_linear on the packed form of
 * W_sup at that level (bit for bit when both take the same kernel family).  `workspace` as for
 * elsa_nm_linear (elsa_workspace_bytes of the same shape and level).
 */
elsa_status elsa_nm_linear_masked(const void* X, int rows, const void* W_sup, const void* bias, int out, int in,
                                  int N, int M, elsa_dtype dtype, void* Y, void* workspace,
                                  size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* One linear module of the per-layer table (Sec. 3: configuration alpha = (s^1 .. s^L)). */
typedef struct {
    const void* X;       /* [rows][in]  device */
    void* Y;             /* [rows][out] device */
    const void* vals;    /* packed values, device */
    const uint32_t* idx; /* packed indices, device; NULL iff N == M */
    const void* bias;    /* [out] device or NULL */
    int rows, in, out, N, M;
} elsa_layer;

/* Scratch for the table with one region per layer: the sum of elsa_workspace_bytes, each rounded up
 * to 256 bytes (host-only arithmetic). */
size_t elsa_vit_workspace_bytes(const elsa_layer* cfg, int n_layers, elsa_dtype dtype);

/*
 * Runs every layer of the table on one stream, each under its own level N:M (Sec. 3, layer-wise
 * configuration alpha).  `cfg` is a HOST array.  The table is validated as a whole before the
 * first launch; on an error nothing has been enqueued and elsa_last_error() names the layer.
 * The layers of a table must be independent of one another (no layer's X is another layer's Y):
 * given elsa_vit_workspace_bytes(...) of scratch the library builds all weight images first and
 * lets the layers of each kernel family share persistent launches, so their tiles interleave.
 * With less scratch -- at least the largest single elsa_workspace_bytes of the table -- the layers
 * run one after the other through the same region.  Dependent layers go through elsa_nm_linear.
 */
elsa_status elsa_vit_linears(const elsa_layer* cfg, int n_layers, elsa_dtype dtype,
                             void* workspace, size_t workspace_bytes, uint32_t* dev_status,
                             void* stream);

/* One layer of the host-memory variant: every tensor pointer is a HOST pointer. */
typedef struct {
    const void* X;    /* [rows][in]  host */
    void* Y;          /* [rows][out] host, written */
    const void* W;    /* [out][in]   host, dense weight */
    const void* bias; /* [out] host or NULL */
    int rows, in, out, N, M;
} elsa_host_layer;

/* Bytes of device memory elsa_vit_linears_host needs for this table (host-only arithmetic). */
size_t elsa_vit_host_device_bytes(const elsa_host_layer* cfg, int n_layers, elsa_dtype dtype);

/*
 * The whole path from host memory (Sec. 3.1 projection, then Sec. 2 product, per layer of the
 * table): for each layer copy W, bias and X to the device, compress W to its level, multiply,
 * and copy Y back.  `device_mem` is caller-owned device memory of at least
 * elsa_vit_host_device_bytes(...) bytes (two slots, so that one layer's copies overlap its
 * neighbours' kernels), 256-byte aligned.  Copies in and out run on two streams the library creates
 * once per device (no device memory is allocated) and are ordered against the kernels on `stream`
 * by events; `stream` itself waits for the last copy out, so with pinned host memory the call
 * returns after enqueue and every Y is valid once `stream` has been synchronised.  One call at a
 * time per device.
 */
elsa_status elsa_vit_linears_host(const elsa_host_layer* cfg, int n_layers, elsa_dtype dtype,
                                  void* device_mem, size_t device_bytes, uint32_t* dev_status,
                                  void* stream);

/*
 * elsa_nm_linear for callers that have no device memory to hand over as workspace.  (The paper
 * has no counterpart: this is a packaging variant of the call above, not a step of the method.)
 *
 * Who needs it: code that runs where allocating is forbidden or would stall the GPU -- the enqueue
 * hook of an inference-runtime plugin, a serving loop whose framework has already reserved all
 * of the device's memory for its own pool (so cudaMalloc fails), or a latency-critical loop that
 * cannot afford the device-wide synchronisation an allocation implies.  Such callers own X, the
 * packed weight, bias and Y, but cannot produce one more scratch buffer.
 *
 * What it does: the same kernels as elsa_nm_linear (tensor-core variant), with the weight image
 * rebuilt in a fixed scratch array that lives inside the library, ELSA_STATIC_SCRATCH_BYTES long.
 * Every GPU on which the library is loaded holds that array until the process exits.  The call
 * itself performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 * Limits and rules
 *   - out * in * 2 must not exceed ELSA_STATIC_SCRATCH_BYTES when N < M (ELSA_ERR_WORKSPACE, with
 *     a message naming both numbers, otherwise).  The dense level N == M needs no scratch and has
 *     no size limit.
 *   - The first call on each device looks up the array's device address (once per device, with
 *     that device current).  Make that first call before starting any stream capture.
 *   - All calls on a device share the one array.  It keeps whatever the previous call left in
 *     it; that is harmless because every call rewrites the whole image it is about to read, so
 *     nothing in it needs clearing.  Two calls whose kernels can overlap on the GPU (different
 *     streams without an ordering between them) race on it: keep them stream-ordered.
 *   - Arguments otherwise as for elsa_nm_linear; the process-wide variant switch is ignored.
 */
#define ELSA_STATIC_SCRATCH_BYTES (8u << 20) /* 8 MiB: up to a 1024 x 4096 16-bit weight */
elsa_status elsa_nm_linear_static(const void* X, int rows, const void* vals, const uint32_t* idx,
                                  const void* bias, int out, int in, int N, int M,
                                  elsa_dtype dtype, void* Y, uint32_t* dev_status, void* stream);

/* Measurement aid: turn the sharing of launches inside elsa_vit_linears off (0) or on (non-zero,
 * the default), process-wide; with it off every layer gets its own launches and its own record
 * in the per-launch timing below. */
void elsa_set_grouping(int on);

/* Test aid: force the kernel variant used by elsa_nm_linear / elsa_vit_linears (process-wide). */
elsa_status elsa_set_linear_variant(elsa_variant v);
elsa_variant elsa_get_linear_variant(void);

/*
 * Per-launch kernel timing, off by default.  Between elsa_profile_start and elsa_profile_stop every
 * kernel the library launches is bracketed by a pair of CUDA events on the stream it is launched
 * on.  elsa_profile_stop synchronises on the recorded events, writes up to `capacity` records in
 * launch order and returns how many launches were recorded (which may exceed `capacity`).
 * Both calls are for single-threaded measurement harnesses.
 */
typedef enum {
    ELSA_KERNEL_COMPRESS = 0,
    ELSA_KERNEL_UNPACK = 1,
    ELSA_KERNEL_LINEAR_SIMT = 2,
    ELSA_KERNEL_LINEAR_TC_DENSE = 3,
    ELSA_KERNEL_LINEAR_TC_PAIR = 4,
    ELSA_KERNEL_NM_TO_SP24 = 5,
    ELSA_KERNEL_LINEAR_TC_SP24 = 6,
    ELSA_KERNEL_LINEAR_TC_SP24_PAIR = 7,
    ELSA_KERNEL_WEIGHT_IMAGES = 8, /* batched unpack / 2-of-4 re-encoding of a table's weights */
    ELSA_KERNEL_LINEAR_TC_SP24_WS = 9, /* 2:4 sparse MMA with the weight block resident in tensor memory */
    ELSA_KERNEL_LINEAR_TC_SP24_ST = 10, /* 2:4 sparse MMA with the weight streaming through tensor memory */
    ELSA_KERNEL_LINEAR_TC_PAIR_I8 = 11, /* INT8 form of the CTA-pair GEMM */
    ELSA_KERNEL_INT8_FORMAT = 12,       /* INT8 compress / unpack */
    ELSA_KERNEL_BLOCK_ROWWISE = 13,     /* LayerNorm, residual add, GELU, column copy of the chained block */
    ELSA_KERNEL_BACKWARD_FORMAT = 14,   /* transposes, column sums and mask of the backward pass */
    ELSA_KERNEL_ATTENTION = 15          /* multi-head self-attention of the chained block */
} elsa_kernel_id;

typedef struct {
    int kernel; /* elsa_kernel_id */
    int layer;  /* index into the table of elsa_vit_linears / _host, -1 for single calls */
    float ms;   /* device time between the two events */
} elsa_kernel_time;

elsa_status elsa_profile_start(void);
int elsa_profile_stop(elsa_kernel_time* records, int capacity);

/* Number of kernels the library has launched from this process so far. */
unsigned long long elsa_launch_count(void);

/* ------------------------------------------------------------------------------------------------
 * INT8 form of the path (paper: Table 6, the searched N:M models under 8-bit post-training quantisation).
 * The quantiser is not part of this library: the caller supplies signed 8-bit weights and activations and
 * their scales (w_scale[o] per output feature, x_scale for the activation tensor).
 *
 * elsa_nm_compress_i8: Sec. 3.1 / Eq. 1 with saliency |w| on the integers (|-128| = 128), lowest position first
 * among equals; vals[out][in / M * N] are the kept bytes in ascending position, idx is the same log2(M)-bit
 * stream as in the 16-bit form.  elsa_nm_unpack_i8: the dense image, zeros at pruned positions.
 * elsa_nm_linear_i8: Y[r][o] = round16( float(sum_k X[r][k] * Wm[o][k]) * (x_scale * w_scale[o]) + bias[o] ): the sum
 * is exact (int32), the int32 -> float conversion, the two products and the sum are each rounded to nearest
 * in fp32, then one rounding to out_dtype.  bias is out_dtype or NULL.  All pointers are DEVICE pointers
 * owned by the caller, row-major, 16-byte aligned; in % 16 == 0, out % 8 == 0.  workspace: at least
 * elsa_workspace_bytes_i8 (0 for N == M), 256-byte aligned.  Asynchronous on `stream`; errors as elsa_nm_linear.
 */
size_t elsa_nm_values_bytes_i8(int out, int in, int N, int M);
size_t elsa_workspace_bytes_i8(int out, int in, int N, int M);
elsa_status elsa_nm_compress_i8(const int8_t* W, int out, int in, int N, int M, int8_t* vals, uint32_t* idx, void* stream);
elsa_status elsa_nm_unpack_i8(const int8_t* vals, const uint32_t* idx, int out, int in, int N, int M, int8_t* W_masked,
                              void* stream);
elsa_status elsa_nm_linear_i8(const int8_t* X, int rows, float x_scale, const int8_t* vals, const uint32_t* idx,
                              const float* w_scale, const void* bias, int out, int in, int N, int M, elsa_dtype out_dtype,
                              void* Y, void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Search-side host code (no GPU): cost model, two-step sampling, enumeration of configurations.
 *
 * Paper: Sec. 3 defines a configuration alpha = (s^1 .. s^L), one level s^l of the level set S per linear
 * module (L = 4B: qkv, proj, fc1, fc2 of every block).  Sec. 3.2 and the appendix's settings define the cost
 * F(alpha) as FLOPs (Table 1's figures are multiply-accumulates: only the linear modules scale with N/M, the
 * rest of the network stays dense) and the budget C_upper as 50 % of the dense model's.  Alg. 3 (two-step
 * sampling): cut [C_lower, C_upper] into intervals, draw one uniformly, then draw a configuration whose cost
 * lies in it from the per-layer level probabilities P_t.  Sec. 2 counts the space: 3 levels over 48 modules
 * give 3^48 configurations.
 *
 * All arrays are HOST memory owned by the caller.  A cost table is cost[l * n_levels + s] = cost of layer l at
 * level s, in any unit (multiply-accumulates from elsa_cost_table_macs, or measured microseconds); P has the
 * same shape (non-negative weights, normalised per layer by the callee); a configuration is choice[l] = index
 * into the level set.  Nothing here is asynchronous.
 */
typedef struct { int rows, in, out; } elsa_linear_shape; /* rows = tokens the module processes */
typedef struct { int N, M; } elsa_level;

/* cost[l][s] = rows * in * out * N_s / M_s multiply-accumulates (Sec. 2: only kept weights are multiplied). */
elsa_status elsa_cost_table_macs(const elsa_linear_shape* layers, int n_layers, const elsa_level* levels, int n_levels,
                                 double* cost);
/* F(alpha) = fixed_cost + sum over layers of cost[l][choice[l]]; fixed_cost carries the part of the network
 * that is never pruned (attention products, patch embedding, head).  -1 on invalid arguments. */
double elsa_config_cost(const double* cost, int n_layers, int n_levels, const int* choice, double fixed_cost);
/*
 * Alg. 3.  Costs are quantised to multiples of `quantum` (> 0; at most 2^22 quanta over the whole range).
 * C_lower is the cost of the cheapest configuration; the n_intervals intervals have equal width, are half
 * open, and the last also contains C_upper (configurations with F <= C_upper take part, Sec. 3.2).
 * uniforms: 1 + n_layers numbers in [0, 1): the first picks the interval, number 1 + l picks the level of layer
 * l by inverse CDF over the levels in their given order, under the distribution of Alg. 3's second step: P_t
 * restricted to the configurations of the interval (computed exactly, without rejection).  Writes choice[l]
 * and, if not NULL, *interval.  ELSA_ERR_SHAPE when the interval holds no configuration of non-zero
 * probability, when C_upper is below C_lower, or when an argument is out of range.
 */
elsa_status elsa_two_step_sample(const double* cost, int n_layers, int n_levels, const double* P, double fixed_cost,
                                 double c_upper, int n_intervals, double quantum, const double* uniforms, int* choice,
                                 int* interval);
/* mass[i] = probability, under P alone, that a configuration's cost falls into interval i of the same cut. */
elsa_status elsa_interval_masses(const double* cost, int n_layers, int n_levels, const double* P, double fixed_cost,
                                 double c_upper, int n_intervals, double quantum, double* mass);
/* n_levels ^ n_layers as a decimal string (Sec. 2's 3^48); returns its length, -1 if `out` is too small. */
int elsa_search_space_size(int n_layers, int n_levels, char* out, size_t capacity);
/* Configuration number `index_decimal` (a decimal string below n_levels ^ n_layers): digit l of the index in base
 * n_levels is the level of layer l. */
elsa_status elsa_config_from_index(const char* index_decimal, int n_layers, int n_levels, int* choice);

/* ------------------------------------------------------------------------------------------------
 * The chained transformer block around the four pruned linears (Sec. 3: the modules qkv, proj, fc1 and fc2 of
 * every block each take one N:M level; Sec. 4.2 quotes the speed of whole models).  The block is the pre-norm
 * ViT block:
 *     x1 = LayerNorm1(x)        qkv = Linear_qkv(x1)        a = attention(qkv)
 *     x2 = x + Linear_proj(a)   x3 = LayerNorm2(x2)         h = GELU(Linear_fc1(x3))    y = x2 + Linear_fc2(h)
 * LayerNorm runs over the `dim` features of a token row (biased variance, eps inside the square root, gain and
 * bias per feature); GELU is the exact form v * Phi(v).  Statistics, bias, activation and residual are computed
 * in fp32 and every tensor that crosses a stage boundary is rounded once to `dtype` (where a linear runs on a
 * kernel whose epilogue cannot take the residual, its output is rounded before the residual is added).
 * Attention: the paper prunes the linear modules and leaves the attention products dense.  Three ways to run it:
 * elsa_vit_block_attn runs the whole block with the library's multi-head self-attention (elsa_attention:
 * a = softmax(q k^T / sqrt d) v per image and head over the image's own tokens, no mask; at most 256 tokens per
 * image, head dimension 64, i.e. the ViT / DeiT shapes; windowed attention with a position bias, as in Swin, is not
 * built); elsa_vit_block_qkv runs the block up to qkv, the caller's own attention turns qkv into a [rows][dim] in
 * region A, and elsa_vit_block_rest runs the block from proj on; elsa_vit_block runs both halves with the stand-in
 * a = V (columns 2 dim .. 3 dim of qkv copied through), which times the linear and elementwise path alone and does
 * not compute a transformer block's attention.
 *
 * All pointers are DEVICE pointers, 16-byte aligned; dim and mlp_dim multiples of 8 and of every M in use.
 * Weights are the packed forms elsa_nm_compress writes: qkv [3 dim][dim], proj [dim][dim], fc1 [mlp_dim][dim],
 * fc2 [dim][mlp_dim].  `scratch`: caller-owned, 256-byte aligned, elsa_vit_block_scratch_bytes(...) bytes; the
 * intermediates stay there after the call at the byte offsets that call reports, in the order of
 * elsa_block_region (region T is the unfused linears' output before the residual; WORKSPACE holds the weight
 * images).  y may not alias x.  Launches are asynchronous on `stream` (weight images are built on a library
 * stream beside the first LayerNorm); errors as for elsa_nm_linear, nothing is enqueued on a validation error.
 */
typedef struct {
    const void* vals;    /* packed values */
    const uint32_t* idx; /* packed indices; NULL iff N == M */
    const void* bias;    /* [out] or NULL */
    int N, M;
} elsa_block_linear;

typedef struct {
    const void* ln1_gain; /* [dim] */
    const void* ln1_bias;
    const void* ln2_gain;
    const void* ln2_bias;
    elsa_block_linear qkv, proj, fc1, fc2;
    float eps;            /* LayerNorm epsilon (1e-6 in DeiT) */
} elsa_block_weights;

typedef enum {
    ELSA_BLOCK_X1 = 0,  /* [rows][dim]     */
    ELSA_BLOCK_QKV = 1, /* [rows][3 dim]   */
    ELSA_BLOCK_A = 2,   /* [rows][dim]     */
    ELSA_BLOCK_X2 = 3,  /* [rows][dim]     */
    ELSA_BLOCK_X3 = 4,  /* [rows][dim]     */
    ELSA_BLOCK_H = 5,   /* [rows][mlp_dim] */
    ELSA_BLOCK_T = 6,   /* [rows][dim]     */
    ELSA_BLOCK_WORKSPACE = 7,
    ELSA_BLOCK_REGIONS = 8
} elsa_block_region;

/* Bytes of scratch for one block; offsets (may be NULL) receives ELSA_BLOCK_REGIONS byte offsets.  0 on invalid
 * arguments.  Host-only arithmetic. */
size_t elsa_vit_block_scratch_bytes(int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                                    size_t* offsets);
/* x [rows][dim] -> regions X1 and QKV of scratch. */
elsa_status elsa_vit_block_qkv(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w,
                               elsa_dtype dtype, void* scratch, size_t scratch_bytes, uint32_t* dev_status, void* stream);
/* x and region A of scratch (written by the caller's attention) -> y [rows][dim]; fills X2, X3, H. */
elsa_status elsa_vit_block_rest(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w,
                                elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes, uint32_t* dev_status,
                                void* stream);
/* Both, with the stand-in a = V between them. */
elsa_status elsa_vit_block(const void* x, int rows, int dim, int mlp_dim, const elsa_block_weights* w, elsa_dtype dtype,
                           void* y, void* scratch, size_t scratch_bytes, uint32_t* dev_status, void* stream);
/* qkv [images * tokens][3 dim] (q | k | v thirds, heads side by side in each) -> a [images * tokens][dim]; the
 * scores and probabilities stay on chip (fp32 scores, probabilities rounded to `dtype` for the second product, fp32
 * row sums, one rounding of a).  dim = 64 * heads or 32 * heads, tokens <= 256. */
elsa_status elsa_attention(const void* qkv, int images, int tokens, int heads, int dim, elsa_dtype dtype, void* a,
                           uint32_t* dev_status, void* stream);
/* The same over windows of `tokens` consecutive rows with additive tables on the scores (Swin's window attention once
 * the rows are in window order): a = softmax(q k^T / sqrt d + bias[head] + mask[window % n_masks]) v.  bias: fp32
 * [heads][tokens][bias_pitch] (the relative-position bias as a dense table), mask: fp32 [n_masks][tokens][bias_pitch] or
 * NULL (the seam mask of shifted windows, one table per window position of an image); rows of bias_pitch >= tokens floats,
 * bias_pitch a multiple of 4, tables 16-byte aligned.  Head dimension 32 or 64 (dim = heads * 32 or heads * 64), tokens <= 256. */
elsa_status elsa_window_attention(const void* qkv, int windows, int tokens, int heads, int dim, const float* bias,
                                  int bias_pitch, const float* mask, int n_masks, elsa_dtype dtype, void* a,
                                  uint32_t* dev_status, void* stream);
/*
 * The Swin form of the block (Table 1 and Fig. 10 of the paper evaluate Swin-S / Swin-B): tokens are an H x W grid per
 * image, attention runs inside windows of window x window tokens of the grid rolled by -shift (shift = 0 or, in every
 * second block, window / 2), with the relative-position bias and, for shift > 0, the seam mask on the scores.  The
 * first LayerNorm writes its rows in window order, qkv, attention and proj work on windows as runs of rows, and the
 * residual add brings proj's rows back to the grid's order.  Regions X1, QKV, A and T of scratch are therefore in
 * window order.  rel_bias: fp32 [heads][window^2][bias_pitch], device; mask: fp32 [(H / window) (W / window)]
 * [window^2][bias_pitch], device, as elsa_swin_mask writes it (required iff shift > 0); bias_pitch a multiple of 4.  dim = 32 or 64 times heads.
 * Patch merging between stages is a separate linear and not part of this call.
 * pack: windows per attention item (1, or more while pack * window^2 <= 256; consecutive windows are consecutive rows,
 * so an item of `pack` windows is a run of rows too, and the 128-row tiles of the tensor cores are better filled: 2 for
 * 7 x 7 windows).  The tables are then per group of windows, [heads][pack window^2][bias_pitch] with -30000 between
 * tokens of different windows (elsa_swin_pack_bias builds it) and [windows of an image / pack][pack window^2][bias_pitch].
 */
typedef struct {
    int H, W, window, shift;
    const float* rel_bias;
    const float* mask;
    int bias_pitch;
    int pack;
} elsa_swin_attn;
/* HOST arithmetic: fills mask [windows of an image / pack][pack window^2][pitch] (host memory) with 0 / -100 and
 * returns the number of tables, -1 on invalid arguments (needs 0 < shift < window). */
int elsa_swin_mask(int H, int W, int window, int shift, int pack, int pitch, float* mask);
/* HOST arithmetic: rel_bias [heads][window^2][window^2] -> packed [heads][pack window^2][pitch], the bias on the
 * diagonal blocks and -30000 elsewhere.  0, or -1 on invalid arguments. */
int elsa_swin_pack_bias(const float* rel_bias, int heads, int window, int pack, int pitch, float* packed);
elsa_status elsa_swin_block(const void* x, int images, int heads, int dim, int mlp_dim, const elsa_block_weights* w,
                            const elsa_swin_attn* attn, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                            uint32_t* dev_status, void* stream);
/* The whole block with elsa_attention between the halves; rows = images * tokens. */
elsa_status elsa_vit_block_attn(const void* x, int images, int tokens, int heads, int dim, int mlp_dim,
                                const elsa_block_weights* w, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                                uint32_t* dev_status, void* stream);
/*
 * n_blocks such blocks in a row (`blocks`: HOST array, one level table per block: the paper's configuration alpha
 * over the whole encoder), optionally followed by the model's final LayerNorm (final_gain / final_bias: [dim] device,
 * or both NULL).  Same results, bit for bit, as n_blocks calls of elsa_vit_block_attn; where a block's last linear runs
 * on a kernel that cannot add the residual, the next block's first LayerNorm (or the final one) adds it in the same
 * pass instead of a kernel of its own.  scratch: elsa_vit_encoder_scratch_bytes(...) bytes, 256-byte aligned (the
 * largest block's scratch plus two activation buffers); y [images * tokens][dim] may not alias x.  All blocks are
 * validated before the first launch.
 */
size_t elsa_vit_encoder_scratch_bytes(int images, int tokens, int dim, int mlp_dim, const elsa_block_weights* blocks,
                                      int n_blocks, elsa_dtype dtype);
elsa_status elsa_vit_encoder(const void* x, int images, int tokens, int heads, int dim, int mlp_dim,
                             const elsa_block_weights* blocks, int n_blocks, const void* final_gain, const void* final_bias,
                             float final_eps, elsa_dtype dtype, void* y, void* scratch, size_t scratch_bytes,
                             uint32_t* dev_status, void* stream);

/* ------------------------------------------------------------------------------------------------
 * Backward pass of the masked linear (Alg. 2, supernet training: the gradient is taken with respect to the
 * sparse weights W(alpha) derived from the shared weight and applied to the shared weight).  For
 * Y = X Wm^T + b with Wm = mask .* W and dY the gradient arriving at Y:
 *     dX [rows][in]  = dY Wm
 *     dW [out][in]   = mask .* (dY^T X)   dense, exact zeros at pruned positions (a pruned weight takes no part
 *                                         in the product; the paper states no straight-through estimator)
 *     db [out]       = sum over rows of dY
 * fp32 accumulation, one rounding to `dtype` per output.  Any of dX, dW, db may be NULL (not computed); vals is
 * needed for dX, X for dW; idx names the kept positions (NULL iff N == M).  All DEVICE pointers, 16-byte aligned;
 * workspace: elsa_backward_workspace_bytes(...) bytes, 256-byte aligned (the transposed masked weight for dX,
 * partial column sums for db).  Both contractions run at the dense rate: the 2:4 sparse MMA needs the zeros along
 * the reduction, which in dX runs over `out`.  Asynchronous on `stream`.
 */
size_t elsa_backward_workspace_bytes(int rows, int in, int out, int N, int M, elsa_dtype dtype);
elsa_status elsa_nm_linear_backward(const void* dY, const void* X, int rows, const void* vals, const uint32_t* idx,
                                    int out, int in, int N, int M, elsa_dtype dtype, void* dX, void* dW, void* db,
                                    void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream);

/*
 * Test hook for the device-side failure path.  Every wait of the tensor-core kernels is bounded: a wait that
 * runs out records ELSA_ERR_TIMEOUT | site << 8 in dev_status and the kernel winds down instead of hanging.
 * This call launches one warp that runs that same wait on a barrier nobody arrives at, with `limit_ns`
 * (1 ns .. 100 ms) in place of the kernels' two seconds; after synchronising, *dev_status holds
 * ELSA_ERR_TIMEOUT | 15 << 8 (if it was 0 before) and the device is usable as before.  dev_status: device
 * pointer, required.  Asynchronous on `stream`.  The paper has no counterpart; it exists for the tests.
 */
elsa_status elsa_selftest_wait_timeout(unsigned long long limit_ns, uint32_t* dev_status, void* stream);

/* Message describing the calling thread's last non-OK status ("" if none). */
const char* elsa_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* ELSA_H */
