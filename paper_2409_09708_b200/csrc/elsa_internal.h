// Internal declarations shared by the translation units of libelsa (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "elsa.h"

namespace elsa {

// log2(M) for the supported group sizes, -1 otherwise.
inline int index_bits(int M) { return M == 4 ? 2 : M == 8 ? 3 : M == 16 ? 4 : -1; }
inline size_t values_per_row(int in, int N, int M) { return (size_t)(in / M) * (size_t)N; }
inline size_t index_words_per_row(int in, int N, int M)
{
    if (N == M) return 0;
    return ((size_t)(in / M) * (size_t)N * (size_t)index_bits(M) + 31) / 32;
}
inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Records a message for elsa_last_error() and returns `st`.
elsa_status fail(elsa_status st, const char* fmt, ...);
// Counts one kernel launch and converts the launch's cudaError_t.
elsa_status launched(const char* what);

// Brackets one kernel launch with CUDA events while profiling is on (see elsa_profile_start).
class ProfileScope {
public:
    ProfileScope(int kernel, cudaStream_t stream);
    ~ProfileScope();
private:
    int slot_;
    cudaStream_t stream_;
};
// Layer index attached to the records of the calling thread (-1 outside a table).
void set_profile_layer(int layer);

#ifdef __CUDACC__
// Programmatic dependent launch.  Every kernel of the library is launched with the attribute that
// lets it start while its predecessor on the stream is still draining; in exchange each kernel calls
// pdl_wait_for_predecessors() before its first access to global memory (it returns once the
// predecessor grid has completed and its writes are visible) and pdl_release_successors() as soon as
// its own successor may begin its set-up.  With a predecessor launched the ordinary way both are no-ops.
__device__ __forceinline__ void pdl_wait_for_predecessors() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release_successors() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                       unsigned cluster_x, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cudaLaunchAttribute attr[2];
    int n = 0;
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
    if (cluster_x > 1) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x;
        attr[n].val.clusterDim.y = 1;
        attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = (unsigned)n;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<Args&&>(args)...);
}
#endif

struct DeviceInfo {
    int device;
    int sm_count;
    int cc_major;
    size_t smem_optin;
};
// Properties of the current device (cached per device).
elsa_status device_info(DeviceInfo* info);

// --- kernels (each enqueues on `stream` and returns the launch status) ---
elsa_status launch_compress(const uint16_t* W, int out, int in, int N, int M, uint16_t* vals,
                            uint32_t* idx, cudaStream_t stream);
elsa_status launch_unpack(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                          uint16_t* Wm, cudaStream_t stream);
elsa_status launch_linear_simt(const uint16_t* X, int rows, const uint16_t* vals,
                               const uint32_t* idx, const uint16_t* bias, int out, int in, int N,
                               int M, elsa_dtype dtype, uint16_t* Y, cudaStream_t stream);
// Dense tensor-core GEMM Y = X Wd^T + bias with Wd a dense [out][in] image (tcgen05 / TMEM / TMA).
elsa_status launch_linear_tc_dense(const uint16_t* X, int rows, const uint16_t* Wd,
                                   const uint16_t* bias, int out, int in, elsa_dtype dtype,
                                   uint16_t* Y, uint32_t* dev_status, cudaStream_t stream);

// The same GEMM on CTA pairs (cluster of two, tcgen05 cta_group::2); for large row counts.
elsa_status launch_linear_tc_pair(const uint16_t* X, int rows, const uint16_t* Wd, const uint16_t* bias,
                                  int out, int in, elsa_dtype dtype, uint16_t* Y, uint32_t* dev_status,
                                  cudaStream_t stream);
// Y [m][n] = A^T B on the same kernel with both operands stored reduction-outermost, A [k][m] and B [k][n]
// (m, n multiples of 8): the weight-gradient product dY^T X without transposed copies.
// With splits > 1 the reduction is cut into that many ranges whose fp32 sums go to partial [splits][m][n] (Y is then
// not written); linear_tc_pair_tn_splits says how many ranges keep the SM pairs occupied.
int linear_tc_pair_tn_splits(int m, int n, int k, int sm_count);
elsa_status launch_linear_tc_pair_tn(const uint16_t* A, const uint16_t* B, int m, int n, int k, elsa_dtype dtype,
                                     uint16_t* Y, int splits, float* partial, uint32_t* dev_status, cudaStream_t stream);
// Levels with N <= 2 on the hardware 2:4 sparse MMA: re-encodes the packed weight into `workspace`
// (2-of-4 values + metadata), then runs the sparse GEMM.
elsa_status launch_linear_tc_sparse(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                    const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype,
                                    uint16_t* Y, void* workspace, uint32_t* dev_status, cudaStream_t stream);
// Forms of the 2-of-4 image (its rows are rounded up to 32, rows past `out` are zero):
//   SP24_ROWS      [row][in/2], row r holds feature r                       (TMA-fed kernels)
//   SP24_PERMUTED  [row][in/2], row r of every block of 32 holds feature 8 * (r % 4) + r / 4 of the block: the
//                  lane order of the kernels whose epilogue transposes with stmatrix (weight-stationary)
//   SP24_TILED     permuted rows, and per (block of 32 rows, 256 k) the 16-byte units of all rows interleaved,
//                  [unit][row][16 bytes], so that a warp reads one unit of 32 rows as one contiguous run
//                  (streaming kernel); needs in % 128 == 0
enum Sp24Layout { SP24_ROWS = 0, SP24_PERMUTED = 1, SP24_TILED = 2 };
// packed weight -> 2-of-4 image + metadata blocks of 2 KB per (128 features, block_k of K), block_k = 64 or 128.
elsa_status launch_nm_to_sp24(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M, int block_k,
                              int layout, uint16_t* a_img, uint8_t* meta, cudaStream_t stream);
// Where the metadata blocks start in a layer's scratch: after the image, whose rows are rounded up to 32.
inline size_t sp24_meta_offset(int out, int in) { return round_up((size_t)((out + 31) / 32 * 32) * (size_t)in, 256); }
// The same on CTA pairs (256 features x 224 rows per pair, K blocks of 128).
elsa_status launch_linear_tc_sparse_pair(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                         const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype,
                                         uint16_t* Y, void* workspace, uint32_t* dev_status, cudaStream_t stream);
// Several N <= 2 layers in one persistent launch of the sparse pair kernel; each job's workspace must
// already hold its re-encoded weight (launch_linear_tc_sparse_pair_prepare).
struct SparseJob {
    const uint16_t* X;
    const uint16_t* bias;
    uint16_t* Y;
    const void* workspace;
    int rows, in, out;
    int act = 0;      // epilogue activation: 0 none, 1 GELU (weight-stationary and streaming kernels only)
};
int linear_tc_sparse_pair_group_max();
elsa_status launch_linear_tc_sparse_pair_prepare(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                                                 int layout, void* workspace, cudaStream_t stream);
elsa_status launch_linear_tc_sparse_pair_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                               cudaStream_t stream);
bool linear_tc_sparse_suits(int in, int N);
// The same product with the 256-feature weight block of each CTA pair resident in tensor memory for a
// whole layer (in % 128 == 0, in <= 1024); jobs as for the pair kernel, same re-encoded weight.
int linear_tc_sparse_ws_group_max();
bool linear_tc_sparse_ws_suits(int in, int out, int N, int sm_count);
elsa_status launch_linear_tc_sparse_ws_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                             cudaStream_t stream);
elsa_status launch_linear_tc_sparse_ws(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                       const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype, uint16_t* Y,
                                       void* workspace, uint32_t* dev_status, cudaStream_t stream);
size_t linear_tc_sparse_workspace(int out, int in);
// The same product with the weight block streaming through tensor memory in K chunks of 256 (in % 128 == 0,
// any length); jobs as for the pair kernel, weight image in the SP24_TILED form.
int linear_tc_sparse_st_group_max();
bool linear_tc_sparse_st_suits(int in, int N);
elsa_status launch_linear_tc_sparse_st_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                             cudaStream_t stream);
elsa_status launch_linear_tc_sparse_st(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                       const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype, uint16_t* Y,
                                       void* workspace, uint32_t* dev_status, cudaStream_t stream);
// Row-wise and elementwise kernels of the chained block (16-bit tensors, fp32 arithmetic, one rounding).
// R == NULL: Yn = LayerNorm(A).  R != NULL: S = A + R, and Yn = LayerNorm(S) unless Yn is NULL.  dim % 8 == 0.
// row_map (or NULL): Swin's window order of the token rows (grid H x W, windows of ws x ws, roll by shift), applied
// to where A is read (on_input) or where Yn is written (on_output).
struct RowMap {
    int H, W, ws, shift;
    int on_input, on_output;
};
elsa_status launch_layer_norm(const uint16_t* A, const uint16_t* R, uint16_t* S, const uint16_t* gain,
                              const uint16_t* beta, uint16_t* Yn, int rows, int dim, float eps, elsa_dtype dtype,
                              cudaStream_t stream, const RowMap* row_map = nullptr);
// Y = act(Y) over `count` values (count % 8 == 0); act as in the GEMM epilogues.
elsa_status launch_act_inplace(uint16_t* Y, long long count, int act, elsa_dtype dtype, cudaStream_t stream);
// dst[r][0 .. cols) = src[r][col0 .. col0 + cols); src rows of src_ld values; all multiples of 8.
elsa_status launch_copy_columns(const uint16_t* src, uint16_t* dst, int rows, int src_ld, int col0, int cols,
                                cudaStream_t stream);
// Multi-head self-attention a = softmax(q k^T / sqrt d + bias + mask) v per image and head on tcgen05 (tokens <= 256,
// head dimension 64 or 32): qkv [images * tokens][3 * dim] -> out [images * tokens][dim].  bias (or NULL):
// fp32 [heads][tokens][bias_pitch]; mask (or NULL): fp32 [n_masks][tokens][bias_pitch], image i takes table i % n_masks.
bool attention_suits(int tokens, int heads, int dim);
elsa_status launch_attention(const uint16_t* qkv, int images, int tokens, int heads, int dim, elsa_dtype dtype,
                             uint16_t* out, uint32_t* dev_status, cudaStream_t stream, const float* bias = nullptr,
                             const float* mask = nullptr, int n_masks = 0, int bias_pitch = 0);
// Operand forms of the backward pass.  transpose16: src [R][C] -> dst [C][Rp] with the tail R..Rp zero (C, Rp
// multiples of 8).  colsum: db [C] = column sums of src [R][C], through ceil(R / 512) * C floats of scratch.
elsa_status launch_transpose16(const uint16_t* src, uint16_t* dst, int R, int C, int Rp, cudaStream_t stream);
elsa_status launch_colsum(const uint16_t* src, int R, int C, float* partial, uint16_t* db, elsa_dtype dtype, cudaStream_t stream);
// Zeroes the pruned positions of a dense [out][in] tensor in place.
elsa_status launch_mask_apply(uint16_t* dW, const uint32_t* idx, int out, int in, int N, int M, cudaStream_t stream);
// dW [out][in] = mask .* round16(sum over ranges of partial [splits][out][in]); idx NULL (N == M) keeps everything.
elsa_status launch_wgrad_finish(const float* partial, int splits, const uint32_t* idx, int out, int in, int N, int M,
                                elsa_dtype dtype, uint16_t* dW, cudaStream_t stream);
// Several levels of one weight in one pass, and the dense projections used by the mask-on-load linear.
constexpr int kMaxLevels = 16;
struct LevelTable {
    int n;
    int N[kMaxLevels];
    uint16_t* vals[kMaxLevels];
    uint32_t* idx[kMaxLevels];
};
elsa_status launch_compress_levels(const uint16_t* W, int out, int in, int M, const LevelTable& t, cudaStream_t stream);
elsa_status launch_mask(const uint16_t* W, int out, int in, int N, int M, uint16_t* Wm, cudaStream_t stream);
elsa_status launch_dense_to_sp24(const uint16_t* W, int out, int in, int N, int M, int block_k, int layout,
                                 uint16_t* a_img, uint8_t* meta, cudaStream_t stream);

// Batched weight-format kernels: one launch over a table of weights (kernel-parameter space).
enum BatchKind { BATCH_COMPRESS = 0, BATCH_UNPACK = 1, BATCH_TO_SP24 = 2 };
struct BatchItem {
    const void* src;
    const void* src2;
    void* dst;
    void* dst2;
    long long first_unit;   // prefix sum of work units over the table
    int out, in, N, M, wpr, aux, aux2, aux3, kind;
};
constexpr int kBatchMax = 256;
struct BatchTable {
    BatchItem item[kBatchMax];
    long long total_units;
    int n;
};
void batch_add_compress(BatchTable* t, const uint16_t* W, int out, int in, int N, int M, uint16_t* vals, uint32_t* idx);
void batch_add_unpack(BatchTable* t, const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                      uint16_t* Wm);
void batch_add_to_sp24(BatchTable* t, const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                       int block_k, int layout, uint16_t* a_img, uint8_t* meta);
elsa_status launch_compress_batch(const BatchTable& t, cudaStream_t stream);
elsa_status launch_image_batch(const BatchTable& t, cudaStream_t stream);

// Several dense-rate layers in one persistent launch of the CTA-pair kernel (at most
// linear_tc_pair_group_max() of them): their tiles form one sequence.
struct PairJob {
    const uint16_t* X;
    const uint16_t* Wd;     // dense weight image [out][in]
    const uint16_t* bias;
    uint16_t* Y;
    int rows, in, out;
    const float* w_scale = nullptr;   // INT8 form only
    float x_scale = 0.f;
    int act = 0;                          // epilogue activation: 0 none, 1 GELU (applied to acc + bias)
    const uint16_t* residual = nullptr;   // [rows][out], added after the activation, before the one rounding
    int splits = 1;                       // Tn form: ranges the reduction is cut into; > 1 writes fp32 sums to `partial`
    float* partial = nullptr;             // [splits][rows][out]
};
int linear_tc_pair_group_max();
elsa_status launch_linear_tc_pair_group(const PairJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                        cudaStream_t stream);
// INT8 form of the same GEMM: X [rows][in] and the dense weight image Wd [out][in] hold signed 8-bit integers,
// accumulation is int32, Y[r][o] = round16(float(acc) * (x_scale * w_scale[o]) + bias[o]).
elsa_status launch_linear_tc_pair_i8(const int8_t* X, int rows, const int8_t* Wd, const float* w_scale, float x_scale,
                                     const uint16_t* bias, int out, int in, elsa_dtype dtype, uint16_t* Y,
                                     uint32_t* dev_status, cudaStream_t stream);
// Whether the problem has enough 256-row tiles to occupy every SM pair.
bool linear_tc_pair_suits(int rows, int out, int sm_count);

}  // namespace elsa
