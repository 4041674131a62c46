// Helper kernels of the masked linear's backward pass (ELSA, Alg. 2: the gradient is taken with respect to the
// sparse weights derived from the shared weight; for Y = X Wm^T + b that is dX = dY Wm, dW = mask .* dY^T X,
// db = column sums of dY).  The two contractions run on the dense tensor-core GEMM of the forward path, which
// wants both operands with the reduction index contiguous; these kernels bring the operands into that form:
//   transpose16    [R][C] -> [C][Rp] (Rp >= R, the tail zero): the masked weight for dX
//   mask_apply     zeroes the pruned positions of a dense [out][in] gradient in place, from the index stream
//   colsum_partial column sums of dY over chunks of 512 rows; colsum_finish adds the chunks and rounds once
#include "elsa_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace elsa {
namespace {

constexpr int kTile = 64;

template <bool kBf16>
__device__ __forceinline__ float to_float(uint16_t u)
{
    if constexpr (kBf16) return __uint_as_float((uint32_t)u << 16);
    else return __half2float(__ushort_as_half(u));
}

template <bool kBf16>
__device__ __forceinline__ uint16_t from_float(float f)
{
    if constexpr (kBf16) return __bfloat16_as_ushort(__float2bfloat16_rn(f));
    else return __half_as_ushort(__float2half_rn(f));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4])
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void stmatrix_x4_transposed(uint32_t addr, const uint32_t (&r)[4])
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};"
                 :: "r"(addr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]) : "memory");
}

// One block per 64 x 64 tile.  src [R][C] (C % 8 == 0), dst [C][Rp] (Rp % 8 == 0).  The tile is read with
// 16-byte loads into shared memory, transposed there in 8 x 8 blocks (ldmatrix, stmatrix.trans; rows of
// 144 bytes keep both free of bank conflicts) and written with 16-byte stores.  Blocks of the last tile row also
// write the zero tail R..Rp of their dst rows.
__global__ void __launch_bounds__(256)
transpose16_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int R, int C, int Rp)
{
    constexpr int kPitch = kTile + 8;   // values per shared-memory row
    __shared__ __align__(16) uint16_t tile_in[kTile][kPitch];
    __shared__ __align__(16) uint16_t tile_out[kTile][kPitch];
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int r0 = blockIdx.x * kTile, c0 = blockIdx.y * kTile;   // row tiles on x: their count has no 65535 limit
    const int t = threadIdx.x;
    // load: 64 rows x 8 vectors of 8 values (rows past R and columns past C as zeros)
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int slot = t + 256 * i;
        const int r = slot >> 3, v = slot & 7;
        uint4 u = make_uint4(0u, 0u, 0u, 0u);
        if (r0 + r < R && c0 + 8 * v < C)
            u = __ldg(reinterpret_cast<const uint4*>(src + (size_t)(r0 + r) * (size_t)C + c0 + 8 * v));
        *reinterpret_cast<uint4*>(&tile_in[r][8 * v]) = u;
    }
    __syncthreads();
    {
        // warp w transposes the eight 8 x 8 blocks of source rows 8w .. 8w + 7
        const int w = t >> 5, lane = t & 31;
        const uint32_t in_base = (uint32_t)__cvta_generic_to_shared(&tile_in[0][0]);
        const uint32_t out_base = (uint32_t)__cvta_generic_to_shared(&tile_out[0][0]);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int j = 4 * half + (lane >> 3);               // column block this lane addresses
            uint32_t r[4];
            ldmatrix_x4(in_base + (uint32_t)(((8 * w + (lane & 7)) * kPitch + 8 * j) * 2), r);
            stmatrix_x4_transposed(out_base + (uint32_t)(((8 * j + (lane & 7)) * kPitch + 8 * w) * 2), r);
        }
    }
    __syncthreads();
    // store: 64 dst rows (source columns) x 8 vectors of 8 source rows
    const bool last = blockIdx.x == gridDim.x - 1;
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const int slot = t + 256 * i;
        const int c = slot >> 3, v = slot & 7;
        if (c0 + c >= C) continue;
        uint16_t* row = dst + (size_t)(c0 + c) * (size_t)Rp;
        if (r0 + 8 * v < Rp) *reinterpret_cast<uint4*>(row + r0 + 8 * v) = *reinterpret_cast<const uint4*>(&tile_out[c][8 * v]);
        if (last)
            for (int r = r0 + kTile + 8 * v; r < Rp; r += kTile) *reinterpret_cast<uint4*>(row + r) = make_uint4(0u, 0u, 0u, 0u);
    }
}

// partial[chunk][c] = sum of src[r][c] over the chunk's rows (kColsumRows per chunk).  A block covers 256 columns:
// 32 threads across (eight columns each, one 16-byte load per row) by 8 threads down; every thread adds its rows
// in ascending order, the eight row lanes are added in a fixed order, so the result does not depend on timing.
constexpr int kColsumRows = 512;

template <bool kBf16>
__global__ void __launch_bounds__(256)
colsum_partial_kernel(const uint16_t* __restrict__ src, int R, int C, float* __restrict__ partial)
{
    __shared__ float acc[8][256 + 8];
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int c = blockIdx.y * 256 + 8 * tx;
    const int r_begin = blockIdx.x * kColsumRows;
    const int r_end = min(R, r_begin + kColsumRows);
    float s[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (c < C) {
        for (int r = r_begin + ty; r < r_end; r += 8) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * (size_t)C + c));
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                s[2 * q] += to_float<kBf16>((uint16_t)(w[q] & 0xffffu));
                s[2 * q + 1] += to_float<kBf16>((uint16_t)(w[q] >> 16));
            }
        }
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[ty][8 * tx + e] = s[e];
    __syncthreads();
    const int col = blockIdx.y * 256 + threadIdx.x;
    if (col < C) {
        float t = 0.f;
#pragma unroll
        for (int y = 0; y < 8; ++y) t += acc[y][threadIdx.x];
        partial[(size_t)blockIdx.x * (size_t)C + col] = t;
    }
}

// db[c] = round16(sum over tiles of partial[tile][c]), tiles in ascending order.
template <bool kBf16>
__global__ void __launch_bounds__(256) colsum_finish_kernel(const float* __restrict__ partial, int tiles, int C, uint16_t* __restrict__ db)
{
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= C) return;
    float s = 0.f;
    for (int i = 0; i < tiles; ++i) s += partial[(size_t)i * (size_t)C + c];
    db[c] = from_float<kBf16>(s);
}

// One thread per group of M: keeps the N positions the index stream names, zeroes the rest.
template <int M>
__global__ void __launch_bounds__(256)
mask_apply_kernel(uint16_t* __restrict__ dW, const uint32_t* __restrict__ idx, int out, int in, int N, int words_per_row)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int groups_per_row = in / M;
    if (gid >= (long long)out * groups_per_row) return;
    const int o = (int)(gid / groups_per_row), g = (int)(gid % groups_per_row);
    const uint32_t* row = idx + (size_t)o * (size_t)words_per_row;
    uint32_t keep = 0;
    for (int t = 0; t < N; ++t) {
        const int bit = (g * N + t) * B;
        const int w = bit >> 5, sh = bit & 31;
        uint32_t f = row[w] >> sh;
        if (sh + B > 32) f |= row[w + 1] << (32 - sh);
        keep |= 1u << (f & (M - 1));
    }
    uint32_t* p = reinterpret_cast<uint32_t*>(dW + (size_t)o * (size_t)in + (size_t)g * M);
#pragma unroll
    for (int q = 0; q < M / 2; ++q) {
        const uint32_t m = ((keep >> (2 * q)) & 1u ? 0x0000ffffu : 0u) | ((keep >> (2 * q + 1)) & 1u ? 0xffff0000u : 0u);
        if (m != 0xffffffffu) p[q] &= m;
    }
}

// One thread per group of M weights: adds the ranges' fp32 sums in ascending order, rounds once, zeroes what the
// index stream does not keep (everything is kept when idx is NULL).
template <int M, bool kBf16>
__global__ void __launch_bounds__(256)
wgrad_finish_kernel(const float* __restrict__ partial, int splits, const uint32_t* __restrict__ idx, int out, int in, int N,
                    int words_per_row, uint16_t* __restrict__ dW)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const int groups_per_row = in / M;
    if (gid >= (long long)out * groups_per_row) return;
    const int o = (int)(gid / groups_per_row), g = (int)(gid % groups_per_row);
    uint32_t keep = 0xffffffffu;
    if (idx != nullptr) {
        keep = 0;
        const uint32_t* row = idx + (size_t)o * (size_t)words_per_row;
        for (int t = 0; t < N; ++t) {
            const int bit = (g * N + t) * B;
            const int w = bit >> 5, sh = bit & 31;
            uint32_t f = row[w] >> sh;
            if (sh + B > 32) f |= row[w + 1] << (32 - sh);
            keep |= 1u << (f & (M - 1));
        }
    }
    const size_t at = (size_t)o * (size_t)in + (size_t)g * M;
    const size_t plane = (size_t)out * (size_t)in;
    float acc[M];
#pragma unroll
    for (int q = 0; q < M / 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(partial + at + 4 * q);
        acc[4 * q] = v.x; acc[4 * q + 1] = v.y; acc[4 * q + 2] = v.z; acc[4 * q + 3] = v.w;
    }
    for (int s = 1; s < splits; ++s) {
#pragma unroll
        for (int q = 0; q < M / 4; ++q) {
            const float4 v = *reinterpret_cast<const float4*>(partial + (size_t)s * plane + at + 4 * q);
            acc[4 * q] += v.x; acc[4 * q + 1] += v.y; acc[4 * q + 2] += v.z; acc[4 * q + 3] += v.w;
        }
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(dW + at);
#pragma unroll
    for (int q = 0; q < M / 2; ++q) {
        const uint32_t lo = (keep >> (2 * q)) & 1u ? from_float<kBf16>(acc[2 * q]) : 0u;
        const uint32_t hi = (keep >> (2 * q + 1)) & 1u ? from_float<kBf16>(acc[2 * q + 1]) : 0u;
        dst[q] = lo | (hi << 16);
    }
}

}  // namespace

elsa_status launch_colsum_finish(const float* partial, int tiles, int C, uint16_t* db, elsa_dtype dtype, cudaStream_t stream);

elsa_status launch_transpose16(const uint16_t* src, uint16_t* dst, int R, int C, int Rp, cudaStream_t stream)
{
    if (R <= 0 || C <= 0) return ELSA_OK;
    const dim3 grid((unsigned)((R + kTile - 1) / kTile), (unsigned)((C + kTile - 1) / kTile));
    ProfileScope scope(ELSA_KERNEL_BACKWARD_FORMAT, stream);
    launch_pdl(transpose16_kernel, grid, dim3(256), 0, stream, 1, src, dst, R, C, Rp);
    return launched("transpose16");
}

// db [C] = column sums of src [R][C]; partial: ceil(R / 512) * C floats of scratch.
elsa_status launch_colsum(const uint16_t* src, int R, int C, float* partial, uint16_t* db, elsa_dtype dtype, cudaStream_t stream)
{
    const int chunks = (R + kColsumRows - 1) / kColsumRows;
    {
        const dim3 grid((unsigned)chunks, (unsigned)((C + 255) / 256));
        ProfileScope scope(ELSA_KERNEL_BACKWARD_FORMAT, stream);
        if (dtype == ELSA_BF16) launch_pdl(colsum_partial_kernel<true>, grid, dim3(256), 0, stream, 1, src, R, C, partial);
        else launch_pdl(colsum_partial_kernel<false>, grid, dim3(256), 0, stream, 1, src, R, C, partial);
        elsa_status st = launched("colsum_partial");
        if (st != ELSA_OK) return st;
    }
    return launch_colsum_finish(partial, chunks, C, db, dtype, stream);
}

elsa_status launch_colsum_finish(const float* partial, int tiles, int C, uint16_t* db, elsa_dtype dtype, cudaStream_t stream)
{
    const unsigned grid = (unsigned)((C + 255) / 256);
    ProfileScope scope(ELSA_KERNEL_BACKWARD_FORMAT, stream);
    if (dtype == ELSA_BF16) launch_pdl(colsum_finish_kernel<true>, dim3(grid), dim3(256), 0, stream, 1, partial, tiles, C, db);
    else launch_pdl(colsum_finish_kernel<false>, dim3(grid), dim3(256), 0, stream, 1, partial, tiles, C, db);
    return launched("colsum_finish");
}

elsa_status launch_wgrad_finish(const float* partial, int splits, const uint32_t* idx, int out, int in, int N, int M,
                                elsa_dtype dtype, uint16_t* dW, cudaStream_t stream)
{
    const long long groups = (long long)out * (in / M);
    const unsigned grid = (unsigned)((groups + 255) / 256);
    const int wpr = (int)index_words_per_row(in, N, M);
    const uint32_t* ix = N == M ? nullptr : idx;
    const bool bf = dtype == ELSA_BF16;
    ProfileScope scope(ELSA_KERNEL_BACKWARD_FORMAT, stream);
#define ELSA_FINISH(MM)                                                                                                     \
    do {                                                                                                                  \
        if (bf) launch_pdl(wgrad_finish_kernel<MM, true>, dim3(grid), dim3(256), 0, stream, 1, partial, splits, ix, out, in, N, wpr, dW); \
        else launch_pdl(wgrad_finish_kernel<MM, false>, dim3(grid), dim3(256), 0, stream, 1, partial, splits, ix, out, in, N, wpr, dW);   \
    } while (0)
    if (M == 4) ELSA_FINISH(4);
    else if (M == 8) ELSA_FINISH(8);
    else ELSA_FINISH(16);
#undef ELSA_FINISH
    return launched("wgrad_finish");
}

elsa_status launch_mask_apply(uint16_t* dW, const uint32_t* idx, int out, int in, int N, int M, cudaStream_t stream)
{
    if (N == M) return ELSA_OK;
    const long long groups = (long long)out * (in / M);
    const unsigned grid = (unsigned)((groups + 255) / 256);
    const int wpr = (int)index_words_per_row(in, N, M);
    ProfileScope scope(ELSA_KERNEL_BACKWARD_FORMAT, stream);
    if (M == 4) launch_pdl(mask_apply_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, dW, idx, out, in, N, wpr);
    else if (M == 8) launch_pdl(mask_apply_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, dW, idx, out, in, N, wpr);
    else launch_pdl(mask_apply_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, dW, idx, out, in, N, wpr);
    return launched("mask_apply");
}

}  // namespace elsa
