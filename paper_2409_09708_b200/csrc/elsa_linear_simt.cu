// CUDA-core N:M sparse linear that reads the packed form directly: for every kept weight the
// index field selects the activation it multiplies (Sec. 2, Fig. 2 bottom of the ELSA paper: decode
// the index, pick the matching activation, multiply-accumulate only the kept weights).
//
// This variant exists so that the tensor-core variants can be cross-checked against a kernel
// with a different data path; it is not tuned and is never chosen automatically.

#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "elsa_internal.h"

namespace elsa {
namespace {

template <bool kBf16>
__device__ __forceinline__ float to_float(uint16_t u)
{
    if constexpr (kBf16) return __bfloat162float(__ushort_as_bfloat16(u));
    else return __half2float(__ushort_as_half(u));
}

template <bool kBf16>
__device__ __forceinline__ uint16_t from_float(float f)
{
    if constexpr (kBf16) return __bfloat16_as_ushort(__float2bfloat16_rn(f));
    else return __half_as_ushort(__float2half_rn(f));
}

template <bool kBf16>
__global__ void __launch_bounds__(256)
linear_simt_kernel(const uint16_t* __restrict__ X, int rows, const uint16_t* __restrict__ vals,
                   const uint32_t* __restrict__ idx, const uint16_t* __restrict__ bias, int out, int in,
                   int N, int M, int B, int words_per_row, uint16_t* __restrict__ Y)
{
    const int o = blockIdx.x * 32 + threadIdx.x;
    const int r = blockIdx.y * 8 + threadIdx.y;
    if (o >= out || r >= rows) return;

    const int groups = in / M;
    const uint16_t* x = X + (size_t)r * in;
    const uint16_t* v = vals + (size_t)o * ((size_t)groups * N);
    const uint32_t* row_idx = words_per_row ? idx + (size_t)o * words_per_row : nullptr;

    float acc = 0.f;
    for (int g = 0; g < groups; ++g) {
        for (int t = 0; t < N; ++t) {
            const int field = g * N + t;
            int pos = t;  // N == M: every position kept, in order
            if (row_idx) {
                const int bit = field * B;
                const int w = bit >> 5, sh = bit & 31;
                uint32_t f = row_idx[w] >> sh;
                if (sh + B > 32) f |= row_idx[w + 1] << (32 - sh);
                pos = (int)(f & (uint32_t)(M - 1));
            }
            acc = fmaf(to_float<kBf16>(x[g * M + pos]), to_float<kBf16>(v[field]), acc);
        }
    }
    if (bias) acc += to_float<kBf16>(bias[o]);
    Y[(size_t)r * out + o] = from_float<kBf16>(acc);
}

}  // namespace

elsa_status launch_linear_simt(const uint16_t* X, int rows, const uint16_t* vals,
                               const uint32_t* idx, const uint16_t* bias, int out, int in, int N,
                               int M, elsa_dtype dtype, uint16_t* Y, cudaStream_t stream)
{
    const dim3 block(32, 8);
    const dim3 grid((out + 31) / 32, (rows + 7) / 8);
    const int B = index_bits(M);
    const int wpr = (int)index_words_per_row(in, N, M);
    if (grid.y > 65535u) return fail(ELSA_ERR_SHAPE, "SIMT variant supports at most 524280 rows");
    ProfileScope scope(ELSA_KERNEL_LINEAR_SIMT, stream);
    if (dtype == ELSA_BF16)
        linear_simt_kernel<true><<<grid, block, 0, stream>>>(X, rows, vals, idx, bias, out, in, N, M,
                                                             B, wpr, Y);
    else
        linear_simt_kernel<false><<<grid, block, 0, stream>>>(X, rows, vals, idx, bias, out, in, N, M,
                                                              B, wpr, Y);
    return launched("linear_simt");
}

}  // namespace elsa
