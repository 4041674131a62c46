// Device code of the weight-format kernels, shared by the per-weight launches and the batched ones:
// N:M projection + packing (Sec. 3.1 / Eq. 1 and the compressed form of Sec. 1 / Sec. 2 of the ELSA
// paper), its inverse, and the re-encoding of a packed weight as 2-of-4 values + tensor-memory
// metadata for the sparse MMA.  Each function handles one unit of work given its global index.
#pragma once

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
// Ranks of the M magnitudes of one group, 4 bits each: rank_i = #{j : |w_j| > |w_i|} + #{j < i : |w_j| == |w_i|}
// (larger magnitude first, lower position first among equals).  Magnitudes are compared as the 15 low
// bits of the pattern.  The level N keeps exactly the elements with rank < N, for every N at once.
template <int M>
__device__ __forceinline__ unsigned long long group_ranks(const uint16_t (&w)[M])
{
    unsigned long long ranks = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const uint32_t ki = w[i] & 0x7FFFu;
        int rank = 0;
#pragma unroll
        for (int j = 0; j < M; ++j) {
            const uint32_t kj = w[j] & 0x7FFFu;
            rank += (kj > ki) || (j < i && kj == ki);
        }
        ranks |= (unsigned long long)rank << (4 * i);
    }
    return ranks;
}

template <int M>
__device__ __forceinline__ uint32_t keep_mask(unsigned long long ranks, int N)
{
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) keep |= (uint32_t)((int)((ranks >> (4 * i)) & 15ull) < N) << i;
    return keep;
}

// One warp compresses 32 consecutive groups of one row, one group per lane, to each of `n_levels`
// levels N_list[l]:M (one read of W, ranks computed once).  The 32 groups own exactly N*b whole index
// words of the row's bitstream, so the warp assembles its words in shared memory and writes them with
// one coalesced store.
template <int M>
__device__ __forceinline__ void compress_segment_levels(const uint16_t* __restrict__ W, int in, int n_levels,
                                                        const int* N_list, uint16_t* const* vals_list,
                                                        uint32_t* const* idx_list, int segs_per_row, long long seg_id,
                                                        uint32_t (*words)[kMaxIndexWordsPerSegment])
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;

    const int o = (int)(seg_id / segs_per_row);
    const int seg = (int)(seg_id % segs_per_row);
    const int groups_per_row = in / M;
    const int g = seg * 32 + lane;
    const bool valid = g < groups_per_row;

    uint16_t w[M];
    unsigned long long ranks = 0;
    if (valid) {
        load_group<M>(W + (size_t)o * in + (size_t)g * M, w);
        ranks = group_ranks<M>(w);
    }

    for (int l = 0; l < n_levels; ++l) {
        const int N = N_list[l];
        uint16_t* vals = vals_list[l];
        uint32_t* idx = idx_list[l];
        const int words_per_row = (N == M) ? 0 : (groups_per_row * N * B + 31) / 32;
        const int seg_words = N * B;  // index words this segment owns (when N < M)

        if (words_per_row) {
            for (int k = lane; k < seg_words; k += 32) words[warp][k] = 0;
            __syncwarp();
        }
        if (valid) {
            const uint32_t keep = keep_mask<M>(ranks, N);
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
            for (int k = lane; k < seg_words && first + k < words_per_row; k += 32) row[first + k] = words[warp][k];
            __syncwarp();
        }
    }
}

// ---- single-level fast path for M = 4 and M = 8 (the levels of the ViT tables) -------------------
//
// Same result as compress_segment_levels with one level, in about a third of the instructions:
//   * every position gets a unique key (magnitude bits above, M-1-position below), so "the N of largest
//     magnitude, lowest position first among equals" is "key >= the N-th largest key";
//   * the N-th largest key comes from a sorting network (5 / 19 compare-exchanges);
//   * kept values are compacted with byte permutes driven by a small table in shared memory: for each
//     keep mask, the kept positions in ascending order as 4-bit fields (the permute selectors) and as
//     log2(M)-bit fields (the index bits to store);
//   * one vector store per group for the values.
struct CompactEntry { uint32_t order4; uint32_t fields; };

template <int M>
__device__ __forceinline__ void build_compact_table(CompactEntry* table)
{
    constexpr int B = (M == 4) ? 2 : 3;
    for (int m = threadIdx.x; m < (1 << M); m += blockDim.x) {
        uint32_t o4 = 0, f = 0;
        int t = 0;
        for (int i = 0; i < M; ++i)
            if ((m >> i) & 1) { o4 |= (uint32_t)i << (4 * t); f |= (uint32_t)i << (B * t); ++t; }
        table[m].order4 = o4;
        table[m].fields = f;
    }
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel)
{
    uint32_t r;
    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
    return r;
}

__device__ __forceinline__ void sort2_desc(uint32_t& a, uint32_t& b)
{
    const uint32_t hi = max(a, b), lo = min(a, b);
    a = hi; b = lo;
}

// Keep mask of one group: bit i set iff position i is among the N kept.  h[] are the 16-bit patterns.
template <int M>
__device__ __forceinline__ uint32_t keep_mask_sorted(const uint32_t (&h)[M], int N)
{
    constexpr int S = (M == 4) ? 2 : 3;
    uint32_t k[M], s[M];
#pragma unroll
    for (int i = 0; i < M; ++i) { k[i] = ((h[i] & 0x7FFFu) << S) | (uint32_t)(M - 1 - i); s[i] = k[i]; }
    if constexpr (M == 8) {
        // The levels of the ViT tables need less than a full sort.  Keys are unique and carry their position
        // in the low bits, so the one or two largest keys name the kept positions directly; for N = 4 two
        // sorted halves give the 4th largest without merging them.
        if (N <= 2) {
            sort2_desc(s[0], s[1]); sort2_desc(s[2], s[3]); sort2_desc(s[4], s[5]); sort2_desc(s[6], s[7]);
            // top two of each half from two sorted pairs, then of the whole group
            const uint32_t a0 = max(s[0], s[2]), a1 = max(min(s[0], s[2]), max(s[1], s[3]));
            const uint32_t b0 = max(s[4], s[6]), b1 = max(min(s[4], s[6]), max(s[5], s[7]));
            const uint32_t top = max(a0, b0), second = max(min(a0, b0), max(a1, b1));
            uint32_t keep = 1u << (7u - (top & 7u));
            if (N == 2) keep |= 1u << (7u - (second & 7u));
            return keep;
        }
        if (N == 4) {
            sort2_desc(s[0], s[1]); sort2_desc(s[2], s[3]); sort2_desc(s[4], s[5]); sort2_desc(s[6], s[7]);
            sort2_desc(s[0], s[2]); sort2_desc(s[1], s[3]); sort2_desc(s[4], s[6]); sort2_desc(s[5], s[7]);
            sort2_desc(s[1], s[2]); sort2_desc(s[5], s[6]);
            // i elements of one half and j of the other lie above min(a_i, b_j): with i + j = 2 it is at most the
            // 4th largest, and so are a_3 and b_3 (a half that supplies all four); the largest candidate is it
            const uint32_t thr4 = max(max(max(s[3], s[7]), min(s[0], s[6])), max(min(s[1], s[5]), min(s[2], s[4])));
            uint32_t keep4 = 0;
#pragma unroll
            for (int i = 0; i < M; ++i) keep4 |= (k[i] >= thr4 ? 1u : 0u) << i;
            return keep4;
        }
    }
    if constexpr (M == 4) {
        sort2_desc(s[0], s[1]); sort2_desc(s[2], s[3]);
        sort2_desc(s[0], s[2]); sort2_desc(s[1], s[3]);
        sort2_desc(s[1], s[2]);
    } else {
        sort2_desc(s[0], s[1]); sort2_desc(s[2], s[3]); sort2_desc(s[4], s[5]); sort2_desc(s[6], s[7]);
        sort2_desc(s[0], s[2]); sort2_desc(s[1], s[3]); sort2_desc(s[4], s[6]); sort2_desc(s[5], s[7]);
        sort2_desc(s[1], s[2]); sort2_desc(s[5], s[6]);
        sort2_desc(s[0], s[4]); sort2_desc(s[1], s[5]); sort2_desc(s[2], s[6]); sort2_desc(s[3], s[7]);
        sort2_desc(s[2], s[4]); sort2_desc(s[3], s[5]);
        sort2_desc(s[1], s[2]); sort2_desc(s[3], s[4]); sort2_desc(s[5], s[6]);
    }
    uint32_t thr = s[0];
#pragma unroll
    for (int t = 1; t < M; ++t) thr = (N > t) ? s[t] : thr;      // the N-th largest key
    uint32_t keep = 0;
#pragma unroll
    for (int i = 0; i < M; ++i) keep |= (k[i] >= thr ? 1u : 0u) << i;
    return keep;
}

// Split in two so that a warp can have the loads of several segments in flight before it works on the
// first: one 16-byte load per lane is too little outstanding memory traffic to cover its own latency.
template <int M>
__device__ __forceinline__ void compress_fast_load(const uint16_t* __restrict__ W, int in, int o, int seg,
                                                   uint32_t (&r)[M / 2])
{
    constexpr int R = M / 2;                      // 32-bit registers per group
    const int lane = threadIdx.x & 31;
    const int g = seg * 32 + lane;
#pragma unroll
    for (int q = 0; q < R; ++q) r[q] = 0;
    if (g < in / M) {
        const uint16_t* src = W + (size_t)o * in + (size_t)g * M;
        if constexpr (M == 4) { const uint2 v = *reinterpret_cast<const uint2*>(src); r[0] = v.x; r[1] = v.y; }
        else { const uint4 v = *reinterpret_cast<const uint4*>(src); r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w; }
    }
}

// NC: the level's N as a compile-time constant (0 = take `N_runtime`): with N known every branch on it folds.
template <int M, int NC>
__device__ __forceinline__ void compress_fast_emit(const uint32_t (&r)[M / 2], int in, int N_runtime,
                                                   uint16_t* __restrict__ vals, uint32_t* __restrict__ idx,
                                                   int o, int seg,
                                                   uint32_t (*words)[kMaxIndexWordsPerSegment],
                                                   const CompactEntry* table)
{
    static_assert(M == 4 || M == 8, "fast path for groups of 4 and 8");
    constexpr int B = (M == 4) ? 2 : 3;
    constexpr int R = M / 2;
    const int N = NC ? NC : N_runtime;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int groups_per_row = in / M;
    const int g = seg * 32 + lane;
    const bool valid = g < groups_per_row;
    const int words_per_row = (N == M) ? 0 : (groups_per_row * N * B + 31) / 32;
    const int seg_words = N * B;

    uint16_t* dst = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
    if (N == M) {                                 // dense level: the values are the weight
        if (valid) {
            if constexpr (M == 4) *reinterpret_cast<uint2*>(dst) = make_uint2(r[0], r[1]);
            else *reinterpret_cast<uint4*>(dst) = make_uint4(r[0], r[1], r[2], r[3]);
        }
        return;
    }
    for (int k = lane; k < seg_words; k += 32) words[warp][k] = 0;
    __syncwarp();
    if (valid) {
        uint32_t h[M];
#pragma unroll
        for (int q = 0; q < R; ++q) { h[2 * q] = r[q] & 0xFFFFu; h[2 * q + 1] = r[q] >> 16; }
        const uint32_t keep = keep_mask_sorted<M>(h, N);
        const CompactEntry e = table[keep];
        // low and high bytes of the halfwords as two planes, compacted by the position list, re-interleaved
        uint32_t w[R];
        if constexpr (M == 4) {
            const uint32_t lo = prmt(prmt(r[0], r[1], 0x6420u), 0u, e.order4);
            const uint32_t hi = prmt(prmt(r[0], r[1], 0x7531u), 0u, e.order4);
            w[0] = prmt(lo, hi, 0x5140u);
            w[1] = prmt(lo, hi, 0x7362u);
        } else {
            const uint32_t l0 = prmt(r[0], r[1], 0x6420u), l1 = prmt(r[2], r[3], 0x6420u);
            const uint32_t h0 = prmt(r[0], r[1], 0x7531u), h1 = prmt(r[2], r[3], 0x7531u);
            const uint32_t lo03 = prmt(l0, l1, e.order4 & 0xFFFFu), lo47 = prmt(l0, l1, e.order4 >> 16);
            const uint32_t hi03 = prmt(h0, h1, e.order4 & 0xFFFFu), hi47 = prmt(h0, h1, e.order4 >> 16);
            w[0] = prmt(lo03, hi03, 0x5140u);
            w[1] = prmt(lo03, hi03, 0x7362u);
            w[2] = prmt(lo47, hi47, 0x5140u);
            w[3] = prmt(lo47, hi47, 0x7362u);
        }
        // the group's N values are contiguous: the widest store their common alignment allows
        if ((N & 3) == 0) {
            *reinterpret_cast<uint2*>(dst) = make_uint2(w[0], w[1]);          // N = 4 (M = 8)
        } else if ((N & 1) == 0) {
#pragma unroll
            for (int q = 0; q < R; ++q)
                if (q < (N >> 1)) reinterpret_cast<uint32_t*>(dst)[q] = w[q];
        } else {
#pragma unroll
            for (int t = 0; t < M; ++t)
                if (t < N) dst[t] = (uint16_t)(w[t >> 1] >> (16 * (t & 1)));
        }
        // index bits: at most 21 (M = 8) or 6 (M = 4) bits at bit offset lane * N * B of the segment
        const int bit0 = lane * seg_words;
        const int w0 = bit0 >> 5, sh = bit0 & 31;
        const uint32_t lo = e.fields << sh;
        const uint32_t hi = sh ? (e.fields >> (32 - sh)) : 0u;
        if (lo) atomicOr(&words[warp][w0], lo);
        if (hi) atomicOr(&words[warp][w0 + 1], hi);
    }
    __syncwarp();
    const int first = seg * seg_words;
    uint32_t* row = idx + (size_t)o * words_per_row;
    for (int k = lane; k < seg_words && first + k < words_per_row; k += 32) row[first + k] = words[warp][k];
    __syncwarp();
}

template <int M, int NC = 0>
__device__ __forceinline__ void compress_segment_fast(const uint16_t* __restrict__ W, int in, int N,
                                                      uint16_t* __restrict__ vals, uint32_t* __restrict__ idx,
                                                      int segs_per_row, long long seg_id,
                                                      uint32_t (*words)[kMaxIndexWordsPerSegment],
                                                      const CompactEntry* table)
{
    // a weight has far fewer than 2^32 segments: 32-bit division
    const uint32_t o = (uint32_t)seg_id / (uint32_t)segs_per_row;
    const uint32_t seg = (uint32_t)seg_id - o * (uint32_t)segs_per_row;
    uint32_t r[M / 2];
    compress_fast_load<M>(W, in, (int)o, (int)seg, r);
    compress_fast_emit<M, NC>(r, in, N, vals, idx, (int)o, (int)seg, words, table);
}

// The same with the 16 bytes of the group already in registers (requested one unit ahead by the caller).
template <int M, int NC = 0>
__device__ __forceinline__ void compress_segment_fast_preloaded(const uint32_t (&r4)[4], int in, int N,
                                                                uint16_t* __restrict__ vals, uint32_t* __restrict__ idx,
                                                                int o, int seg, uint32_t (*words)[kMaxIndexWordsPerSegment],
                                                                const CompactEntry* table)
{
    uint32_t r[M / 2];
#pragma unroll
    for (int q = 0; q < M / 2; ++q) r[q] = r4[q];
    compress_fast_emit<M, NC>(r, in, N, vals, idx, o, seg, words, table);
}

// Single level: the form elsa_nm_compress uses.
template <int M>
__device__ __forceinline__ void compress_segment(const uint16_t* __restrict__ W, int in, int N,
                                                 uint16_t* __restrict__ vals, uint32_t* __restrict__ idx,
                                                 int segs_per_row, int words_per_row, long long seg_id,
                                                 uint32_t (*words)[kMaxIndexWordsPerSegment])
{
    (void)words_per_row;
    uint16_t* vals_one = vals;
    uint32_t* idx_one = idx;
    compress_segment_levels<M>(W, in, 1, &N, &vals_one, &idx_one, segs_per_row, seg_id, words);
}

// One thread projects one group of the dense weight onto level N:M: kept values stay, the others
// become +0.0 (the "dynamic masking" of Sec. 3.1 applied to the shared weight, with no packed form).
template <int M>
__device__ __forceinline__ void mask_group(const uint16_t* __restrict__ W, int N, uint16_t* __restrict__ Wm, long long gid)
{
    uint16_t w[M];
    load_group<M>(W + (size_t)gid * M, w);
    const uint32_t keep = keep_mask<M>(group_ranks<M>(w), N);
    uint16_t* dst = Wm + (size_t)gid * M;
    if constexpr (M == 4) {
        uint2 r;
        r.x = (keep & 1u ? w[0] : 0u) | ((uint32_t)(keep & 2u ? w[1] : 0u) << 16);
        r.y = (keep & 4u ? w[2] : 0u) | ((uint32_t)(keep & 8u ? w[3] : 0u) << 16);
        *reinterpret_cast<uint2*>(dst) = r;
    } else {
#pragma unroll
        for (int q = 0; q < M / 8; ++q) {
            uint32_t x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int i = 8 * q + 2 * k;
                x[k] = ((keep >> i) & 1u ? (uint32_t)w[i] : 0u) | (((keep >> (i + 1)) & 1u ? (uint32_t)w[i + 1] : 0u) << 16);
            }
            reinterpret_cast<uint4*>(dst)[q] = make_uint4(x[0], x[1], x[2], x[3]);
        }
    }
}

// One thread rebuilds one group: N values scattered to their positions, +0.0 elsewhere.
template <int M>
__device__ __forceinline__ void unpack_group(const uint16_t* __restrict__ vals, const uint32_t* __restrict__ idx,
                                             int in, int N, uint16_t* __restrict__ Wm, int words_per_row,
                                             long long gid)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    const int groups_per_row = in / M;
    const int o = (int)(gid / groups_per_row);
    const int g = (int)(gid % groups_per_row);

    const uint16_t* v = vals + (size_t)o * ((size_t)groups_per_row * N) + (size_t)g * N;
    if constexpr (M != 16) {
        // Groups of 4 and 8 with N < M: the kept values are loaded with the widest access their alignment
        // allows, split into a plane of low bytes and a plane of high bytes, scattered to their positions by
        // byte permutes (selector nibble of position i = slot holding its value; unused positions point at
        // slot M-1, which is zero because N < M), and re-interleaved.
        if (words_per_row) {
            constexpr int R = M / 2;
            const uint32_t* row = idx + (size_t)o * words_per_row;
            const int bit0 = g * N * B;
            const int w0 = bit0 >> 5, sh = bit0 & 31;
            const uint32_t lo = row[w0];
            const uint32_t hi = (sh + N * B > 32) ? row[w0 + 1] : 0u;
            const uint32_t fields = __funnelshift_r(lo, hi, sh);
            uint32_t vr[R];
#pragma unroll
            for (int q = 0; q < R; ++q) vr[q] = 0;
            if ((N & 3) == 0) {                                   // N = 4 (M = 8)
                const uint2 t = *reinterpret_cast<const uint2*>(v);
                vr[0] = t.x; vr[1] = t.y;
            } else if ((N & 1) == 0) {
#pragma unroll
                for (int q = 0; q < R; ++q)
                    if (q < (N >> 1)) vr[q] = reinterpret_cast<const uint32_t*>(v)[q];
            } else {
#pragma unroll
                for (int t = 0; t < M; ++t)
                    if (t < N) vr[t >> 1] |= (uint32_t)v[t] << (16 * (t & 1));
            }
            uint32_t inv = (M == 8) ? 0x77777777u : 0x3333u;
#pragma unroll
            for (int t = 0; t < M - 1; ++t)
                if (t < N) {
                    const uint32_t pos4 = ((fields >> (t * B)) & (uint32_t)(M - 1)) * 4u;
                    inv = (inv & ~(0xFu << pos4)) | ((uint32_t)t << pos4);
                }
            uint16_t* dst = Wm + (size_t)o * in + (size_t)g * M;
            if constexpr (M == 4) {
                const uint32_t pl = prmt(prmt(vr[0], vr[1], 0x6420u), 0u, inv);
                const uint32_t ph = prmt(prmt(vr[0], vr[1], 0x7531u), 0u, inv);
                *reinterpret_cast<uint2*>(dst) = make_uint2(prmt(pl, ph, 0x5140u), prmt(pl, ph, 0x7362u));
            } else {
                const uint32_t l0 = prmt(vr[0], vr[1], 0x6420u), l1 = prmt(vr[2], vr[3], 0x6420u);
                const uint32_t h0 = prmt(vr[0], vr[1], 0x7531u), h1 = prmt(vr[2], vr[3], 0x7531u);
                const uint32_t pl03 = prmt(l0, l1, inv & 0xFFFFu), pl47 = prmt(l0, l1, inv >> 16);
                const uint32_t ph03 = prmt(h0, h1, inv & 0xFFFFu), ph47 = prmt(h0, h1, inv >> 16);
                *reinterpret_cast<uint4*>(dst) = make_uint4(prmt(pl03, ph03, 0x5140u), prmt(pl03, ph03, 0x7362u),
                                                            prmt(pl47, ph47, 0x5140u), prmt(pl47, ph47, 0x7362u));
            }
            return;
        }
    }
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

// One thread per (weight row, 16 consecutive k): rebuilds those 16 positions from the packed form,
// then emits, per aligned chunk of 4, two values with ascending positions (i0 < i1).  Pruned
// positions are zero in the rebuilt segment, so a chunk with fewer than two kept weights simply
// borrows a zero from another position.
// Second half of the 2-of-4 re-encoding: given 16 consecutive positions of a weight row with the pruned
// ones already zero (d) and the kept set (keep), emits two values per aligned chunk of 4 (ascending
// positions, a zero borrowed where fewer than two are kept) and the chunk nibbles as tensor memory wants them.
// In the permuted forms (Sp24Layout) weight row o lands in image row (o & ~31) | (4 * (o % 8) + (o % 32) / 8), so
// that row r of a block of 32 holds feature 8 * (r % 4) + r / 4: the order in which the transposing stores of the
// tensor-memory-fed kernels want the features in tensor-memory lanes.  The tiled form also interleaves the
// 16-byte units of the 32 rows of a block inside every 256 k.  The image has its rows rounded up to 32; rows
// past `out` are written as zeros.
__device__ __forceinline__ void sp24_emit(const uint16_t (&d)[16], uint32_t keep, bool real, int o_src, int seg, int k0, int in,
                                          int out, uint16_t* __restrict__ a_img, uint16_t* __restrict__ meta16, int k_blocks,
                                          int steps_per_block, int layout)
{
    const int o = layout != SP24_ROWS ? ((o_src & ~31) | (4 * (o_src & 7) + ((o_src & 31) >> 3))) : o_src;
    constexpr int kFeatTile = 128;
    uint32_t nibbles = 0;
    uint16_t sel[8];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const uint32_t m4 = (keep >> (4 * c)) & 15u;
        const int cnt = __popc(m4);
        int i0, i1;
        if (cnt >= 2) { i0 = __ffs(m4) - 1; i1 = 31 - __clz(m4); }
        else if (cnt == 1) { const int p = __ffs(m4) - 1; i0 = (p == 3) ? 0 : p; i1 = 3; }
        else { i0 = 0; i1 = 1; }
        nibbles |= (uint32_t)(i0 | (i1 << 2)) << (4 * c);
        uint16_t v0 = d[4 * c], v1 = d[4 * c];
#pragma unroll
        for (int i = 1; i < 4; ++i) {
            v0 = (i == i0) ? d[4 * c + i] : v0;
            v1 = (i == i1) ? d[4 * c + i] : v1;
        }
        sel[2 * c] = v0;
        sel[2 * c + 1] = v1;
    }

    if (k0 < in && o_src < ((out + 31) & ~31)) {      // `d` is all zero where the row or the segment is padding
        uint4 r;
        r.x = sel[0] | ((uint32_t)sel[1] << 16);
        r.y = sel[2] | ((uint32_t)sel[3] << 16);
        r.z = sel[4] | ((uint32_t)sel[5] << 16);
        r.w = sel[6] | ((uint32_t)sel[7] << 16);
        size_t at = (size_t)o * (size_t)in + (size_t)k0;        // byte offset of (row o, k0) in the row-major forms
        if (layout == SP24_TILED)
            at = (size_t)(o >> 5) * 32 * (size_t)in + (size_t)(k0 >> 8) * 8192 + (size_t)((((k0 & 255) >> 4) * 32 + (o & 31)) * 16);
        *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(a_img) + at) = r;
    }
    // metadata half-word: block (feature tile, k block) -> lane -> 4 words, one per K step of 32; a
    // block covers steps_per_block (2 or 4) steps and leaves the other words zero
    const int ftile = o / kFeatTile, m = o % kFeatTile;
    const int kb = seg / (2 * steps_per_block), step = (seg / 2) % steps_per_block, k1 = seg % 2;
    const int lane = (m % 8) + 8 * k1 + 16 * (m / 16);
    const int hi = (m / 8) % 2;
    const size_t word = (((size_t)ftile * k_blocks + kb) * 128 + lane) * 4 + step;
    meta16[2 * word + hi] = (uint16_t)nibbles;
    if (steps_per_block == 2) meta16[2 * (word + 2) + hi] = 0;
}



// One thread per (weight row, 16 consecutive k) of a PACKED weight: rebuilds those 16 positions, then
// emits their 2-of-4 form.
template <int M>
__device__ __forceinline__ void to_sp24_segment(const uint16_t* __restrict__ vals, const uint32_t* __restrict__ idx,
                                                int out, int in, int N, int words_per_row,
                                                uint16_t* __restrict__ a_img, uint16_t* __restrict__ meta16,
                                                int k_blocks, int steps_per_block, int layout, long long tid)
{
    constexpr int B = (M == 4) ? 2 : (M == 8) ? 3 : 4;
    constexpr int G = 16 / M;                         // groups per 16-k segment
    const int segs = k_blocks * steps_per_block * 2;  // 16-k segments per (padded) row
    const int o = (int)(tid / segs);                  // padded row index
    const int seg = (int)(tid % segs);
    const int k0 = seg * 16;

    uint16_t d[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) d[i] = 0;
    uint32_t keep = 0;
    const bool real = o < out && k0 < in;             // in is a multiple of 16 on this path
    if (real) {
        const int groups_per_row = in / M;
        const uint16_t* v = vals + (size_t)o * ((size_t)groups_per_row * N);
        const uint32_t* row = idx + (size_t)o * words_per_row;
#pragma unroll
        for (int gl = 0; gl < G; ++gl) {
            const int g = k0 / M + gl;
            for (int t = 0; t < N; ++t) {
                const long long bit = ((long long)g * N + t) * B;
                const int w0 = (int)(bit >> 5), sh = (int)(bit & 31);
                uint32_t f = row[w0] >> sh;
                if (sh + B > 32) f |= row[w0 + 1] << (32 - sh);
                const int pos = gl * M + (int)(f & (uint32_t)(M - 1));
                const uint16_t val = v[(size_t)g * N + t];
#pragma unroll
                for (int i = 0; i < 16; ++i) d[i] = (i == pos) ? val : d[i];
                keep |= 1u << pos;
            }
        }
    }
    sp24_emit(d, keep, real, o, seg, k0, in, out, a_img, meta16, k_blocks, steps_per_block, layout);
}

// The same from the DENSE shared weight: the 16 positions are projected onto level N:M on the fly
// (N <= 2), so the supernet's forward needs no packed copy of the weight.
template <int M>
__device__ __forceinline__ void dense_to_sp24_segment(const uint16_t* __restrict__ W, int out, int in, int N,
                                                      uint16_t* __restrict__ a_img, uint16_t* __restrict__ meta16,
                                                      int k_blocks, int steps_per_block, int layout, long long tid)
{
    constexpr int G = 16 / M;
    const int segs = k_blocks * steps_per_block * 2;
    const int o = (int)(tid / segs);
    const int seg = (int)(tid % segs);
    const int k0 = seg * 16;

    uint16_t d[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) d[i] = 0;
    uint32_t keep = 0;
    const bool real = o < out && k0 < in;
    if (real) {
#pragma unroll
        for (int gl = 0; gl < G; ++gl) {
            uint16_t w[M];
            load_group<M>(W + (size_t)o * in + k0 + gl * M, w);
            const uint32_t kg = keep_mask<M>(group_ranks<M>(w), N);
#pragma unroll
            for (int i = 0; i < M; ++i) d[gl * M + i] = ((kg >> i) & 1u) ? w[i] : (uint16_t)0;
            keep |= kg << (gl * M);
        }
    }
    sp24_emit(d, keep, real, o, seg, k0, in, out, a_img, meta16, k_blocks, steps_per_block, layout);
}

}  // namespace
}  // namespace elsa
