// N:M projection of a weight matrix and its compressed form, and the inverse.
//
// elsa_nm_compress: Sec. 3.1 / Eq. 1 of the ELSA paper with magnitude saliency (keep the N largest
// |w| of each group of M consecutive weights), written in the compressed form of Sec. 1 / Sec. 2
// (kept values + one log2(M)-bit index each).  Both kernels are plain streaming kernels: one
// 16-byte load per group of eight, integer compares, coalesced word stores.

#include "elsa_internal.h"

namespace elsa {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kMaxIndexWordsPerSegment = 64;  // 32 groups x N*b bits, N*b <= 60 for N < M <= 16

template <int M>
__device__ __forceinline__ void load_group(const uint16_t* p, uint16_t (&w)[M])
{
    if constexpr (M == 4) {
        uint2 v = *reinterpret_cast<const uint2*>(p);
        w[0] = v.x & 0xFFFF; w[1] = v.x >> 16; w[2] = v.y & 0xFFFF; w[3] = v.y >> 16;
    } else {
#pragma unroll
        for (int q = 0; q < M / 8; ++q) {
            uint4 v = reinterpret_cast<const uint4*>(p)[q];
            w[8 * q + 0] = v.x & 0xFFFF; w[8 * q + 1] = v.x >> 16;
            w[8 * q + 2] = v.y & 0xFFFF; w[8 * q + 3] = v.y >> 16;
            w[8 * q + 4] = v.z & 0xFFFF; w[8 * q + 5] = v.z >> 16;
            w[8 * q + 6] = v.w & 0xFFFF; w[8 * q + 7] = v.w >> 16;
        }
    }
}

// One warp compresses 32 consecutive groups of one row, one group per lane.  The 32 groups own
// exactly N*b whole index words of the row's bitstream, so each warp assembles its words in shared
// memory and writes them with one coalesced store.
template <int M>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
nm_compress_kernel(const uint16_t* __restrict__ W, int out, int in, int N, uint16_t* __restrict__ vals,
                   uint32_t* __restrict__ idx, int segs_per_row, int words_per_row)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    __shared__ uint32_t words[kWarpsPerBlock][kMaxIndexWordsPerSegment];

    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const long long seg_id = (long long)blockIdx.x * kWarpsPerBlock + warp;
    const long long total = (long long)out * segs_per_row;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (seg_id >= total) return;  // whole warps leave together; no block-wide barrier is used

    const int o = (int)(seg_id / segs_per_row);
    const int seg = (int)(seg_id % segs_per_row);
    const int groups_per_row = in / M;
    const int g = seg * 32 + lane;
    const bool valid = g < groups_per_row;
    const int seg_words = N * B;  // index words this segment owns (when N < M)

    if (words_per_row) {
        for (int w = lane; w < seg_words; w += 32) words[warp][w] = 0;
        __syncwarp();
    }

    if (valid) {
        uint16_t w[M];
        load_group<M>(W + (size_t)o * in + (size_t)g * M, w);

        // rank_i = #{j : |w_j| > |w_i|} + #{j < i : |w_j| == |w_i|}; keep iff rank_i < N.
        // Magnitudes are compared as the 15 low bits of the pattern.
        uint32_t keep = 0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
            const uint32_t ki = w[i] & 0x7FFFu;
            int rank = 0;
#pragma unroll
            for (int j = 0; j < M; ++j) {
                const uint32_t kj = w[j] & 0x7FFFu;
                rank += (kj > ki) || (j < i && kj == ki);
            }
            keep |= (uint32_t)(rank < N) << i;
        }

        uint16_t* v = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
        unsigned long long fields = 0;
        int t = 0;
#pragma unroll
        for (int i = 0; i < M; ++i) {
            if ((keep >> i) & 1u) {
                v[t] = w[i];
                fields |= (unsigned long long)i << (t * B);
                ++t;
            }
        }

        if (words_per_row) {
            const int bit0 = lane * seg_words;  // bit offset of this group's fields in the segment
            const int w0 = bit0 >> 5, sh = bit0 & 31;
            // up to 60 bits shifted by up to 31: three words at most
            const uint32_t lo = (uint32_t)(fields << sh);
            const uint32_t mid = (uint32_t)(fields >> (32 - sh));
            const uint32_t hi = sh ? (uint32_t)(fields >> (64 - sh)) : 0u;
            // a zero part may lie past the segment's last word and is skipped
            if (lo) atomicOr(&words[warp][w0], lo);
            if (mid) atomicOr(&words[warp][w0 + 1], mid);
            if (hi) atomicOr(&words[warp][w0 + 2], hi);
        }
    }

    if (words_per_row) {
        __syncwarp();
        const int first = seg * seg_words;
        uint32_t* row = idx + (size_t)o * words_per_row;
        for (int w = lane; w < seg_words && first + w < words_per_row; w += 32)
            row[first + w] = words[warp][w];
    }
}

// One thread rebuilds one group: N values scattered to their positions, +0.0 elsewhere.
template <int M>
__global__ void __launch_bounds__(256)
nm_unpack_kernel(const uint16_t* __restrict__ vals, const uint32_t* __restrict__ idx, int out, int in,
                 int N, uint16_t* __restrict__ Wm, int words_per_row)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    const int groups_per_row = in / M;
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (gid >= (long long)out * groups_per_row) return;
    const int o = (int)(gid / groups_per_row);
    const int g = (int)(gid % groups_per_row);

    const uint16_t* v = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
    unsigned long long fields;
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
        fields = 0;  // N == M: position t holds value t
#pragma unroll
        for (int t = 0; t < M; ++t) fields |= (unsigned long long)t << (t * B);
    }

    uint16_t w[M];
#pragma unroll
    for (int i = 0; i < M; ++i) w[i] = 0;
    for (int t = 0; t < N; ++t) {
        const int pos = (int)((fields >> (t * B)) & (M - 1));
        const uint16_t val = v[t];
#pragma unroll
        for (int i = 0; i < M; ++i) w[i] = (i == pos) ? val : w[i];
    }

    uint16_t* dst = Wm + (size_t)o * in + (size_t)g * M;
    if constexpr (M == 4) {
        uint2 r;
        r.x = w[0] | ((uint32_t)w[1] << 16);
        r.y = w[2] | ((uint32_t)w[3] << 16);
        *reinterpret_cast<uint2*>(dst) = r;
    } else {
#pragma unroll
        for (int q = 0; q < M / 8; ++q) {
            uint4 r;
            r.x = w[8 * q + 0] | ((uint32_t)w[8 * q + 1] << 16);
            r.y = w[8 * q + 2] | ((uint32_t)w[8 * q + 3] << 16);
            r.z = w[8 * q + 4] | ((uint32_t)w[8 * q + 5] << 16);
            r.w = w[8 * q + 6] | ((uint32_t)w[8 * q + 7] << 16);
            reinterpret_cast<uint4*>(dst)[q] = r;
        }
    }
}

}  // namespace

elsa_status launch_compress(const uint16_t* W, int out, int in, int N, int M, uint16_t* vals,
                            uint32_t* idx, cudaStream_t stream)
{
    const int groups_per_row = in / M;
    const int segs_per_row = (groups_per_row + 31) / 32;
    const int wpr = (int)index_words_per_row(in, N, M);
    const long long total = (long long)out * segs_per_row;
    const unsigned grid = (unsigned)((total + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const dim3 block(kWarpsPerBlock * 32);
    ProfileScope scope(ELSA_KERNEL_COMPRESS, stream);
    if (M == 4)
        launch_pdl(nm_compress_kernel<4>, dim3(grid), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    else if (M == 8)
        launch_pdl(nm_compress_kernel<8>, dim3(grid), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    else
        launch_pdl(nm_compress_kernel<16>, dim3(grid), block, 0, stream, 1, W, out, in, N, vals, idx, segs_per_row, wpr);
    return launched("nm_compress");
}

elsa_status launch_unpack(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                          uint16_t* Wm, cudaStream_t stream)
{
    const long long total = (long long)out * (in / M);
    const unsigned grid = (unsigned)((total + 255) / 256);
    const int wpr = (int)index_words_per_row(in, N, M);
    ProfileScope scope(ELSA_KERNEL_UNPACK, stream);
    if (M == 4)
        launch_pdl(nm_unpack_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    else if (M == 8)
        launch_pdl(nm_unpack_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    else
        launch_pdl(nm_unpack_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, Wm, wpr);
    return launched("nm_unpack");
}

}  // namespace elsa
