// INT8 form of the N:M path: the same projection, packed form and product on 8-bit integer weights and
// activations (Table 6 of the ELSA paper combines the searched N:M models with 8-bit post-training
// quantisation; the quantiser itself, PTQ4ViT, is outside this library: it supplies the integers and the scales).
//
//   elsa_nm_compress_i8   Sec. 3.1 / Eq. 1 on |w| of int8 weights (|-128| = 128 is the largest magnitude),
//                         lowest position first among equals; kept bytes + the same log2(M)-bit index stream
//   elsa_nm_unpack_i8     the inverse: dense int8 image with zeros at pruned positions
//   elsa_nm_linear_i8     image + tcgen05.mma kind::i8 (int32 accumulators in tensor memory), then
//                         Y = round16(float(acc) * (x_scale * w_scale[o]) + bias[o])
//
// The format kernels are plain streaming kernels (one warp per 32 groups of a row, as the 16-bit general
// path); the GEMM is the CTA-pair kernel of elsa_linear_tc2.cu instantiated for 8-bit operands.

#include "elsa_pack_device.cuh"

namespace elsa {
namespace {

// Keep mask of one group of M int8 weights: rank_i = #{j : |w_j| > |w_i|} + #{j < i : |w_j| == |w_i|}, keep rank < N.
template <int M>
__device__ __forceinline__ uint32_t keep_mask_i8(const int (&w)[M], int N)
{
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const int ki = w[i] < 0 ? -w[i] : w[i];
        int rank = 0;
#pragma unroll
        for (int j = 0; j < M; ++j) {
            const int kj = w[j] < 0 ? -w[j] : w[j];
            rank += (kj > ki) || (j < i && kj == ki);
        }
        keep |= (uint32_t)(rank < N) << i;
    }
    return keep;
}

template <int M>
__device__ __forceinline__ void load_group_i8(const int8_t* p, int (&w)[M])
{
    // groups are M bytes and M-byte aligned (rows are multiples of 16 bytes)
    if constexpr (M == 4) {
        const uint32_t v = *reinterpret_cast<const uint32_t*>(p);
#pragma unroll
        for (int i = 0; i < 4; ++i) w[i] = (int)(int8_t)(v >> (8 * i));
    } else {
#pragma unroll
        for (int q = 0; q < M / 8; ++q) {
            const uint2 v = reinterpret_cast<const uint2*>(p)[q];
#pragma unroll
            for (int i = 0; i < 4; ++i) { w[8 * q + i] = (int)(int8_t)(v.x >> (8 * i)); w[8 * q + 4 + i] = (int)(int8_t)(v.y >> (8 * i)); }
        }
    }
}

// One warp compresses 32 consecutive groups of one row, one group per lane; the 32 groups own exactly N * log2(M)
// whole index words, assembled in shared memory and stored together.
template <int M>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
nm_compress_i8_kernel(const int8_t* __restrict__ W, int out, int in, int N, int8_t* __restrict__ vals,
                      uint32_t* __restrict__ idx, int segs_per_row, int words_per_row)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    __shared__ uint32_t words[kWarpsPerBlock][kMaxIndexWordsPerSegment];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const long long total = (long long)out * segs_per_row;
    const int groups_per_row = in / M;
    const int seg_words = N * B;
    for (long long seg_id = (long long)blockIdx.x * kWarpsPerBlock + warp; seg_id < total;
         seg_id += (long long)gridDim.x * kWarpsPerBlock) {
        const int o = (int)(seg_id / segs_per_row);
        const int seg = (int)(seg_id % segs_per_row);
        const int g = seg * 32 + lane;
        const bool valid = g < groups_per_row;
        if (words_per_row) {
            for (int k = lane; k < seg_words; k += 32) words[warp][k] = 0;
            __syncwarp();
        }
        if (valid) {
            int w[M];
            load_group_i8<M>(W + (size_t)o * in + (size_t)g * M, w);
            const uint32_t keep = N == M ? (M == 16 ? 0xFFFFu : (1u << M) - 1u) : keep_mask_i8<M>(w, N);
            int8_t* v = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
            unsigned long long fields = 0;
            int t = 0;
#pragma unroll
            for (int i = 0; i < M; ++i) {
                if ((keep >> i) & 1u) {
                    v[t] = (int8_t)w[i];
                    fields |= (unsigned long long)i << (t * B);
                    ++t;
                }
            }
            if (words_per_row) {
                const int bit0 = lane * seg_words;
                const int w0 = bit0 >> 5, sh = bit0 & 31;
                const uint32_t lo = (uint32_t)(fields << sh);
                const uint32_t mid = (uint32_t)(fields >> (32 - sh));
                const uint32_t hi = sh ? (uint32_t)(fields >> (64 - sh)) : 0u;
                if (lo) atomicOr(&words[warp][w0], lo);
                if (mid) atomicOr(&words[warp][w0 + 1], mid);
                if (hi) atomicOr(&words[warp][w0 + 2], hi);
            }
        }
        if (words_per_row) {
            __syncwarp();
            const int first = seg * seg_words;
            uint32_t* row = idx + (size_t)o * words_per_row;
            for (int k = lane; k < seg_words && first + k < words_per_row; k += 32) row[first + k] = words[warp][k];
            __syncwarp();
        }
    }
}

// One thread rebuilds one group: N bytes scattered to their positions, zero elsewhere.
template <int M>
__global__ void __launch_bounds__(256)
nm_unpack_i8_kernel(const int8_t* __restrict__ vals, const uint32_t* __restrict__ idx, int out, int in, int N,
                    int8_t* __restrict__ Wm, int words_per_row)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int groups_per_row = in / M;
    if (gid >= (long long)out * groups_per_row) return;
    const int o = (int)(gid / groups_per_row);
    const int g = (int)(gid % groups_per_row);
    const int8_t* v = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
    unsigned long long fields = 0;
    if (words_per_row) {
        const uint32_t* row = idx + (size_t)o * words_per_row;
        const long long bit0 = (long long)g * N * B;
        const int w0 = (int)(bit0 >> 5), sh = (int)(bit0 & 31);
        const int nbits = N * B;
        unsigned long long lo = row[w0];
        if (sh + nbits > 32) lo |= (unsigned long long)row[w0 + 1] << 32;
        fields = lo >> sh;
        if (sh + nbits > 64) fields |= (unsigned long long)row[w0 + 2] << (64 - sh);
    } else {
#pragma unroll
        for (int t = 0; t < M; ++t) fields |= (unsigned long long)t << (t * B);   // N == M: position t holds value t
    }
    uint8_t w[M];
#pragma unroll
    for (int i = 0; i < M; ++i) w[i] = 0;
    for (int t = 0; t < N; ++t) {
        const int pos = (int)((fields >> (t * B)) & (M - 1));
        const uint8_t val = (uint8_t)v[t];
#pragma unroll
        for (int i = 0; i < M; ++i) w[i] = (i == pos) ? val : w[i];
    }
    int8_t* dst = Wm + (size_t)o * in + (size_t)g * M;
#pragma unroll
    for (int q = 0; q < M / 4; ++q)
        reinterpret_cast<uint32_t*>(dst)[q] = (uint32_t)w[4 * q] | ((uint32_t)w[4 * q + 1] << 8) | ((uint32_t)w[4 * q + 2] << 16) |
                                              ((uint32_t)w[4 * q + 3] << 24);
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

elsa_status check_level_i8(int out, int in, int N, int M)
{
    if (out <= 0 || in <= 0) return fail(ELSA_ERR_SHAPE, "non-positive dimension (out=%d, in=%d)", out, in);
    if (index_bits(M) < 0 || N < 1 || N > M) return fail(ELSA_ERR_NM, "unsupported level %d:%d (M in {4, 8, 16}, 1 <= N <= M)", N, M);
    if (in % M != 0) return fail(ELSA_ERR_SHAPE, "in=%d is not a multiple of M=%d", in, M);
    if (in % 16 != 0 || out % 8 != 0)
        return fail(ELSA_ERR_ALIGN, "in=%d must be a multiple of 16 and out=%d of 8 (16-byte row pitches)", in, out);
    return ELSA_OK;
}

elsa_status launch_compress_i8(const int8_t* W, int out, int in, int N, int M, int8_t* vals, uint32_t* idx, cudaStream_t stream)
{
    const int segs_per_row = (in / M + 31) / 32;
    const int wpr = (int)index_words_per_row(in, N, M);
    const long long total = (long long)out * segs_per_row;
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    long long blocks = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > (long long)dev.sm_count * 8) blocks = (long long)dev.sm_count * 8;
    const dim3 block(kWarpsPerBlock * 32);
    ProfileScope scope(ELSA_KERNEL_INT8_FORMAT, stream);
    if (M == 4) launch_pdl(nm_compress_i8_kernel<4>, dim3((unsigned)blocks), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    else if (M == 8) launch_pdl(nm_compress_i8_kernel<8>, dim3((unsigned)blocks), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    else launch_pdl(nm_compress_i8_kernel<16>, dim3((unsigned)blocks), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    return launched("nm_compress_i8");
}

elsa_status launch_unpack_i8(const int8_t* vals, const uint32_t* idx, int out, int in, int N, int M, int8_t* Wm, cudaStream_t stream)
{
    const long long total = (long long)out * (in / M);
    const unsigned grid = (unsigned)((total + 255) / 256);
    const int wpr = (int)index_words_per_row(in, N, M);
    ProfileScope scope(ELSA_KERNEL_INT8_FORMAT, stream);
    if (M == 4) launch_pdl(nm_unpack_i8_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    else if (M == 8) launch_pdl(nm_unpack_i8_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    else launch_pdl(nm_unpack_i8_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    return launched("nm_unpack_i8");
}

}  // namespace
}  // namespace elsa

using namespace elsa;

extern "C" {

size_t elsa_nm_values_bytes_i8(int out, int in, int N, int M)
{
    if (out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    return (size_t)out * values_per_row(in, N, M);
}

size_t elsa_workspace_bytes_i8(int out, int in, int N, int M)
{
    if (out <= 0 || in <= 0 || index_bits(M) < 0 || N < 1 || N > M || in % M != 0) return 0;
    return N == M ? 0 : round_up((size_t)out * (size_t)in, 256);   // the dense int8 image
}

elsa_status elsa_nm_compress_i8(const int8_t* W, int out, int in, int N, int M, int8_t* vals, uint32_t* idx, void* stream)
{
    if (!W || !vals) return fail(ELSA_ERR_NULL, "W and vals must not be NULL");
    elsa_status st = check_level_i8(out, in, N, M);
    if (st != ELSA_OK) return st;
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(W) || !aligned16(vals) || (idx && !aligned16(idx)))
        return fail(ELSA_ERR_ALIGN, "W, vals and idx must be 16-byte aligned");
    return launch_compress_i8(W, out, in, N, M, vals, N == M ? nullptr : idx, (cudaStream_t)stream);
}

elsa_status elsa_nm_unpack_i8(const int8_t* vals, const uint32_t* idx, int out, int in, int N, int M, int8_t* W_masked,
                              void* stream)
{
    if (!vals || !W_masked) return fail(ELSA_ERR_NULL, "vals and W_masked must not be NULL");
    elsa_status st = check_level_i8(out, in, N, M);
    if (st != ELSA_OK) return st;
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(vals) || !aligned16(W_masked) || (idx && !aligned16(idx)))
        return fail(ELSA_ERR_ALIGN, "vals, idx and W_masked must be 16-byte aligned");
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    return launch_unpack_i8(vals, N == M ? nullptr : idx, out, in, N, M, W_masked, (cudaStream_t)stream);
}

elsa_status elsa_nm_linear_i8(const int8_t* X, int rows, float x_scale, const int8_t* vals, const uint32_t* idx,
                              const float* w_scale, const void* bias, int out, int in, int N, int M, elsa_dtype out_dtype,
                              void* Y, void* workspace, size_t workspace_bytes, uint32_t* dev_status, void* stream)
{
    if (!X || !vals || !w_scale || !Y) return fail(ELSA_ERR_NULL, "X, vals, w_scale and Y must not be NULL");
    if (out_dtype != ELSA_F16 && out_dtype != ELSA_BF16) return fail(ELSA_ERR_DTYPE, "out_dtype %d is neither ELSA_F16 nor ELSA_BF16", (int)out_dtype);
    elsa_status st = check_level_i8(out, in, N, M);
    if (st != ELSA_OK) return st;
    if (rows <= 0) return fail(ELSA_ERR_SHAPE, "non-positive rows=%d", rows);
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(X) || !aligned16(vals) || !aligned16(Y) || (idx && !aligned16(idx)) || (bias && !aligned16(bias)) ||
        ((uintptr_t)w_scale & 3u))
        return fail(ELSA_ERR_ALIGN, "X, vals, idx, bias and Y must be 16-byte aligned, w_scale 4-byte aligned");
    const size_t need = elsa_workspace_bytes_i8(out, in, N, M);
    if (need) {
        if (!workspace || workspace_bytes < need)
            return fail(ELSA_ERR_WORKSPACE, "workspace of %zu bytes needed, %zu given", need, workspace ? workspace_bytes : (size_t)0);
        if (((uintptr_t)workspace & 255u) != 0) return fail(ELSA_ERR_ALIGN, "workspace must be 256-byte aligned");
    }
    DeviceInfo dev;
    if ((st = device_info(&dev)) != ELSA_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    const int8_t* Wd = vals;              // the dense level multiplies the stored values as they are
    if (N != M) {
        if ((st = launch_unpack_i8(vals, idx, out, in, N, M, (int8_t*)workspace, s)) != ELSA_OK) return st;
        Wd = (const int8_t*)workspace;
    }
    return launch_linear_tc_pair_i8(X, rows, Wd, w_scale, x_scale, (const uint16_t*)bias, out, in, out_dtype, (uint16_t*)Y,
                                    dev_status, s);
}

}  // extern "C"
