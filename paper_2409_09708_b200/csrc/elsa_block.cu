// Elementwise and row-wise kernels of the transformer block around the four N:M linears (ELSA, Sec. 3: the
// pruned modules qkv, proj, fc1, fc2 sit in the standard pre-norm ViT block; Sec. 4.2 measures whole models):
// LayerNorm, residual add (alone or followed by LayerNorm in the same pass), GELU in place, and the copy of a
// column range.  All of them are HBM-bound streaming kernels: 16-byte loads and stores, fp32 arithmetic, one
// rounding to the 16-bit type per stored value; the row-wise ones give a row to a warp, or, for the model widths
// (128, 256, 512, 768, 1024), several rows at a time to groups of 16 or 32 lanes.
#include "elsa_internal.h"

#include <cuda_bf16.h>
#include <cuda_fp16.h>

namespace elsa {
namespace {

constexpr int kWarpsPerBlock = 8;
constexpr int kCacheVecs = 4;   // 16-byte vectors of a row each lane keeps in registers (rows up to 1024 values)

template <bool kBf16>
__device__ __forceinline__ float2 unpack2(uint32_t u)
{
    if constexpr (kBf16) {
        return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
    } else {
        __half2 h = *reinterpret_cast<__half2*>(&u);
        return __half22float2(h);
    }
}

template <bool kBf16>
__device__ __forceinline__ uint32_t pack2_rn(float a, float b)
{
    if constexpr (kBf16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __half2 v = __floats2half2_rn(a, b);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

template <bool kBf16>
__device__ __forceinline__ void unpack8(const uint4& u, float (&f)[8])
{
    const float2 a = unpack2<kBf16>(u.x), b = unpack2<kBf16>(u.y), c = unpack2<kBf16>(u.z), d = unpack2<kBf16>(u.w);
    f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y; f[4] = c.x; f[5] = c.y; f[6] = d.x; f[7] = d.y;
}

template <bool kBf16>
__device__ __forceinline__ uint4 pack8(const float (&f)[8])
{
    return make_uint4(pack2_rn<kBf16>(f[0], f[1]), pack2_rn<kBf16>(f[2], f[3]), pack2_rn<kBf16>(f[4], f[5]),
                      pack2_rn<kBf16>(f[6], f[7]));
}

// v * Phi(v) = max(v, 0) - 0.5 |v| erfc(|v| / sqrt 2) with erfc as 2^Q(|v|), Q of degree 6: the form and the
// coefficients of the GEMM epilogues (3e-7 absolute error in fp32).
__device__ __forceinline__ float gelu_erf(float v)
{
    const float a = fminf(fabsf(v), 5.9375f);
    float q = fmaf(a, 3.309303065e-05f, -7.692219224e-04f);
    q = fmaf(q, a, 8.080724627e-03f);
    q = fmaf(q, a, -5.341212079e-02f);
    q = fmaf(q, a, -4.587709606e-01f);
    q = fmaf(q, a, -1.151201725e+00f);
    q = fmaf(q, a, 6.939759714e-06f);
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(q));
    return fmaf(-0.5f * fabsf(v), e, fmaxf(v, 0.0f));
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// The row map as the kernels take it: the caller's fields plus what the host can work out once.  Inside an image
// every quotient has a dividend below 2^16 (the host checks H * W), so a division by d is the high half of a product
// with ceil(2^32 / d): exact while dividend * d < 2^32.  With one image's row per 16 or 32 lanes the map's integer
// divisions were most of what a short row's LayerNorm executed.
struct RowMapDev {
    int H, W, ws, shift, on_input, on_output;
    int hw, windows_per_row, ws2;
    uint32_t magic_W, magic_ws;
};

__device__ __forceinline__ int small_div(int n, uint32_t magic, int d)
{
    return d == 1 ? n : (int)__umulhi((uint32_t)n, magic);
}

// Where a row of the token grid goes in window order (Swin): the H x W grid of an image rolled by -shift along both
// axes and cut into ws x ws windows, windows row-major, tokens row-major inside a window.  H == 0: identity.
__device__ __forceinline__ int window_row(const RowMapDev& m, int row)
{
    if (m.H == 0) return row;
    const int b = row / m.hw, t = row - b * m.hw;
    const int i = small_div(t, m.magic_W, m.W), j = t - i * m.W;
    int ir = i - m.shift, jr = j - m.shift;                       // position in the rolled grid (0 <= shift < H, W)
    if (ir < 0) ir += m.H;
    if (jr < 0) jr += m.W;
    const int wi = small_div(ir, m.magic_ws, m.ws), wj = small_div(jr, m.magic_ws, m.ws);
    return b * m.hw + (wi * m.windows_per_row + wj) * m.ws2 + (ir - wi * m.ws) * m.ws + (jr - wj * m.ws);
}

// One warp per row.  map.on_input: A's row r is read at window_row(r) (a tensor in window order brought back to the
// grid's order); map.on_output: Yn's row r is written at window_row(r).  kAdd: the row is S = round16(A + R), written to S (which may be A's or R's own buffer:
// each lane reads its vectors of a row before it writes them).  The statistics are those of the stored 16-bit
// row (for kAdd: of S as rounded), mean first, then the biased variance about it; eps sits inside the root.
// Yn = round16((s - mean) / sqrt(var + eps) * gain + beta), or no normalised output when Yn is NULL.
template <bool kBf16, bool kAdd>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layer_norm_kernel(const uint16_t* A, const uint16_t* R, uint16_t* S, const uint16_t* __restrict__ gain,
                  const uint16_t* __restrict__ beta, uint16_t* Yn, int rows, int dim, float eps, const RowMapDev map)
{
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int lane = threadIdx.x & 31;
    const int vecs = dim >> 3;
    const float inv_dim = 1.0f / (float)dim;
    for (int row = blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); row < rows; row += gridDim.x * kWarpsPerBlock) {
        const int mapped = window_row(map, row);
        const uint4* a4 = reinterpret_cast<const uint4*>(A + (size_t)(map.on_input ? mapped : row) * (size_t)dim);
        const uint4* r4 = kAdd ? reinterpret_cast<const uint4*>(R + (size_t)row * (size_t)dim) : nullptr;
        uint4* s4 = kAdd ? reinterpret_cast<uint4*>(S + (size_t)row * (size_t)dim) : nullptr;
        uint4 cache[kCacheVecs];
        // the row as stored: loaded (and, for kAdd, summed, rounded and written) once
        auto fetch = [&](int v) -> uint4 {
            uint4 u = a4[v];
            if constexpr (kAdd) {
                const uint4 w = r4[v];
                float fa[8], fr[8];
                unpack8<kBf16>(u, fa);
                unpack8<kBf16>(w, fr);
#pragma unroll
                for (int e = 0; e < 8; ++e) fa[e] += fr[e];
                u = pack8<kBf16>(fa);
                s4[v] = u;
            }
            return u;
        };
        // a vector past the register cache is read back from where the row is stored
        auto again = [&](int v) -> uint4 { return kAdd ? s4[v] : a4[v]; };
        float sum = 0.f;
#pragma unroll
        for (int c = 0; c < kCacheVecs; ++c) {
            const int v = lane + 32 * c;
            if (v < vecs) {
                cache[c] = fetch(v);
                float f[8];
                unpack8<kBf16>(cache[c], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) sum += f[e];
            }
        }
        for (int v = lane + 32 * kCacheVecs; v < vecs; v += 32) {
            float f[8];
            unpack8<kBf16>(fetch(v), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) sum += f[e];
        }
        if (Yn == nullptr) continue;
        const float mean = warp_sum(sum) * inv_dim;
        float sq = 0.f;
#pragma unroll
        for (int c = 0; c < kCacheVecs; ++c) {
            if (lane + 32 * c < vecs) {
                float f[8];
                unpack8<kBf16>(cache[c], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) sq += (f[e] - mean) * (f[e] - mean);
            }
        }
        for (int v = lane + 32 * kCacheVecs; v < vecs; v += 32) {
            float f[8];
            unpack8<kBf16>(again(v), f);
#pragma unroll
            for (int e = 0; e < 8; ++e) sq += (f[e] - mean) * (f[e] - mean);
        }
        const float rstd = 1.0f / sqrtf(warp_sum(sq) * inv_dim + eps);
        uint4* y4 = reinterpret_cast<uint4*>(Yn + (size_t)(map.on_output ? mapped : row) * (size_t)dim);
        auto emit = [&](int v, const uint4& u) {
            float f[8], g[8], b[8];
            unpack8<kBf16>(u, f);
            unpack8<kBf16>(__ldg(reinterpret_cast<const uint4*>(gain) + v), g);
            unpack8<kBf16>(__ldg(reinterpret_cast<const uint4*>(beta) + v), b);
#pragma unroll
            for (int e = 0; e < 8; ++e) f[e] = (f[e] - mean) * rstd * g[e] + b[e];
            y4[v] = pack8<kBf16>(f);
        };
#pragma unroll
        for (int c = 0; c < kCacheVecs; ++c)
            if (lane + 32 * c < vecs) emit(lane + 32 * c, cache[c]);
        for (int v = lane + 32 * kCacheVecs; v < vecs; v += 32) emit(v, again(v));
    }
}

// Rows of exactly kLanes * kVpl vectors of eight values (dim = 128, 256, 512, 768, 1024): a group of kLanes lanes owns a row and
// takes kUnroll rows at a time, all of their loads requested before the first is used.  With one row per warp a
// short row leaves (resident warps x row bytes) in flight per SM, a fraction of what the memory latency asks for.
// Same arithmetic per row as layer_norm_kernel (sum, mean, squared deviations about it, one rounding).
template <bool kBf16, bool kAdd, int kLanes, int kVpl, int kUnroll>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
layer_norm_rows_kernel(const uint16_t* A, const uint16_t* R, uint16_t* S, const uint16_t* __restrict__ gain,
                       const uint16_t* __restrict__ beta, uint16_t* Yn, int rows, float eps, const RowMapDev map)
{
    constexpr int kGroups = 32 / kLanes;               // rows side by side in a warp
    constexpr int kRowsPerStep = kGroups * kUnroll;
    constexpr int kDim = kLanes * kVpl * 8;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int lane = threadIdx.x & 31;
    const int sub = lane % kLanes, grp = lane / kLanes;
    const float inv_dim = 1.0f / (float)kDim;
    // this lane's vectors of a row are the same in every row: gain and bias stay in registers
    uint4 g4[kVpl], b4[kVpl];
    if (Yn != nullptr) {
#pragma unroll
        for (int c = 0; c < kVpl; ++c) {
            g4[c] = __ldg(reinterpret_cast<const uint4*>(gain) + sub + kLanes * c);
            b4[c] = __ldg(reinterpret_cast<const uint4*>(beta) + sub + kLanes * c);
        }
    }
    auto group_sum = [&](float v) {
#pragma unroll
        for (int o = kLanes / 2; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        return v;
    };
    const long long steps = ((long long)rows + kRowsPerStep - 1) / kRowsPerStep;
    for (long long step = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); step < steps;
         step += (long long)gridDim.x * kWarpsPerBlock) {
        uint4 x[kUnroll][kVpl];
        int mapped[kUnroll];
        int row_of[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const long long r = step * kRowsPerStep + u * kGroups + grp;
            row_of[u] = r < rows ? (int)r : -1;
            mapped[u] = row_of[u] >= 0 ? window_row(map, row_of[u]) : 0;
        }
        // every load of the step first
        uint4 w[kAdd ? kUnroll : 1][kVpl];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int c = 0; c < kVpl; ++c) {
                x[u][c] = make_uint4(0u, 0u, 0u, 0u);
                if constexpr (kAdd) w[u][c] = make_uint4(0u, 0u, 0u, 0u);
                if (row_of[u] >= 0) {
                    const size_t src = (size_t)(map.on_input ? mapped[u] : row_of[u]) * (size_t)kDim;
                    x[u][c] = reinterpret_cast<const uint4*>(A + src)[sub + kLanes * c];
                    if constexpr (kAdd) w[u][c] = reinterpret_cast<const uint4*>(R + (size_t)row_of[u] * (size_t)kDim)[sub + kLanes * c];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float sum = 0.f;
#pragma unroll
            for (int c = 0; c < kVpl; ++c) {
                float f[8];
                unpack8<kBf16>(x[u][c], f);
                if constexpr (kAdd) {
                    float fr[8];
                    unpack8<kBf16>(w[u][c], fr);
#pragma unroll
                    for (int e = 0; e < 8; ++e) f[e] += fr[e];
                    x[u][c] = pack8<kBf16>(f);
                    if (row_of[u] >= 0) reinterpret_cast<uint4*>(S + (size_t)row_of[u] * (size_t)kDim)[sub + kLanes * c] = x[u][c];
                    unpack8<kBf16>(x[u][c], f);          // the statistics are those of the row as stored
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) sum += f[e];
            }
            if (Yn == nullptr) continue;
            const float mean = group_sum(sum) * inv_dim;
            float sq = 0.f;
#pragma unroll
            for (int c = 0; c < kVpl; ++c) {
                float f[8];
                unpack8<kBf16>(x[u][c], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) sq += (f[e] - mean) * (f[e] - mean);
            }
            const float rstd = 1.0f / sqrtf(group_sum(sq) * inv_dim + eps);
            if (row_of[u] >= 0) {
                uint4* y4 = reinterpret_cast<uint4*>(Yn + (size_t)(map.on_output ? mapped[u] : row_of[u]) * (size_t)kDim);
#pragma unroll
                for (int c = 0; c < kVpl; ++c) {
                    float f[8], g[8], b[8];
                    unpack8<kBf16>(x[u][c], f);
                    unpack8<kBf16>(g4[c], g);
                    unpack8<kBf16>(b4[c], b);
#pragma unroll
                    for (int e = 0; e < 8; ++e) f[e] = (f[e] - mean) * rstd * g[e] + b[e];
                    y4[sub + kLanes * c] = pack8<kBf16>(f);
                }
            }
        }
    }
}

// Y = act(Y) in place, eight values per thread and step.
template <bool kBf16>
__global__ void __launch_bounds__(256) act_inplace_kernel(uint16_t* Y, long long vecs, int act)
{
    pdl_wait_for_predecessors();
    pdl_release_successors();
    uint4* y4 = reinterpret_cast<uint4*>(Y);
    for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < vecs; v += (long long)gridDim.x * blockDim.x) {
        float f[8];
        unpack8<kBf16>(y4[v], f);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            f[e] = act == 1 ? gelu_erf(f[e]) : f[e];
        y4[v] = pack8<kBf16>(f);
    }
}

// dst[r][0 .. cols) = src[r][col0 .. col0 + cols), rows of src_ld values; everything in units of eight values.
__global__ void __launch_bounds__(256)
copy_columns_kernel(const uint16_t* __restrict__ src, uint16_t* __restrict__ dst, int rows, int src_ld, int col0, int cols)
{
    pdl_wait_for_predecessors();
    pdl_release_successors();
    const int vpr = cols >> 3;
    const long long total = (long long)rows * vpr;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
        const int r = (int)(i / vpr), v = (int)(i % vpr);
        reinterpret_cast<uint4*>(dst + (size_t)r * (size_t)cols)[v] =
            __ldg(reinterpret_cast<const uint4*>(src + (size_t)r * (size_t)src_ld + col0) + v);
    }
}

unsigned streaming_grid(long long work_items, int per_block, const DeviceInfo& dev)
{
    long long blocks = (work_items + per_block - 1) / per_block;
    const long long cap = (long long)dev.sm_count * 8;   // one wave of resident blocks; the kernels loop
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (unsigned)blocks;
}

}  // namespace

elsa_status launch_layer_norm(const uint16_t* A, const uint16_t* R, uint16_t* S, const uint16_t* gain,
                              const uint16_t* beta, uint16_t* Yn, int rows, int dim, float eps, elsa_dtype dtype,
                              cudaStream_t stream, const RowMap* row_map)
{
    RowMapDev map = {};
    if (row_map != nullptr && row_map->H != 0) {
        const RowMap& r = *row_map;
        if (r.H < 1 || r.W < 1 || r.ws < 1 || r.H % r.ws != 0 || r.W % r.ws != 0 || r.shift < 0 || r.shift >= r.H ||
            r.shift >= r.W || (long long)r.H * r.W >= 65536)
            return fail(ELSA_ERR_SHAPE, "row map: grid %d x %d, window %d, shift %d", r.H, r.W, r.ws, r.shift);
        map.H = r.H; map.W = r.W; map.ws = r.ws; map.shift = r.shift;
        map.hw = r.H * r.W; map.windows_per_row = r.W / r.ws; map.ws2 = r.ws * r.ws;
        map.magic_W = (uint32_t)(((1ull << 32) + (uint32_t)r.W - 1) / (uint32_t)r.W);
        map.magic_ws = (uint32_t)(((1ull << 32) + (uint32_t)r.ws - 1) / (uint32_t)r.ws);
    }
    if (row_map != nullptr) { map.on_input = row_map->on_input; map.on_output = row_map->on_output; }
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (rows <= 0) return ELSA_OK;
    const dim3 block(kWarpsPerBlock * 32);
    const bool add = R != nullptr;
    ProfileScope scope(ELSA_KERNEL_BLOCK_ROWWISE, stream);
    // the model widths: several rows per warp in flight
#define ELSA_LN_ROWS(LANES, VPL, UNROLL)                                                                                  \
    do {                                                                                                                  \
        const long long steps = ((long long)rows + (32 / LANES) * UNROLL - 1) / ((32 / LANES) * UNROLL);                  \
        const unsigned g = streaming_grid(steps, kWarpsPerBlock, dev);                                                    \
        if (dtype == ELSA_BF16) {                                                                                         \
            if (add) launch_pdl(layer_norm_rows_kernel<true, true, LANES, VPL, UNROLL>, dim3(g), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, eps, map);   \
            else launch_pdl(layer_norm_rows_kernel<true, false, LANES, VPL, UNROLL>, dim3(g), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, eps, map);     \
        } else {                                                                                                          \
            if (add) launch_pdl(layer_norm_rows_kernel<false, true, LANES, VPL, UNROLL>, dim3(g), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, eps, map);  \
            else launch_pdl(layer_norm_rows_kernel<false, false, LANES, VPL, UNROLL>, dim3(g), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, eps, map);    \
        }                                                                                                                 \
        return launched(add ? "residual_add_layer_norm" : "layer_norm");                                                  \
    } while (0)
    if (dim == 128) ELSA_LN_ROWS(16, 1, 4);
    if (dim == 256) ELSA_LN_ROWS(32, 1, 4);
    if (dim == 512) ELSA_LN_ROWS(32, 2, 2);
    if (dim == 1024) ELSA_LN_ROWS(32, 4, 2);
    if (dim == 768) ELSA_LN_ROWS(32, 3, 2);
#undef ELSA_LN_ROWS
    const unsigned grid = streaming_grid(rows, kWarpsPerBlock, dev);
    if (dtype == ELSA_BF16) {
        if (add) launch_pdl(layer_norm_kernel<true, true>, dim3(grid), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, dim, eps, map);
        else launch_pdl(layer_norm_kernel<true, false>, dim3(grid), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, dim, eps, map);
    } else {
        if (add) launch_pdl(layer_norm_kernel<false, true>, dim3(grid), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, dim, eps, map);
        else launch_pdl(layer_norm_kernel<false, false>, dim3(grid), block, 0, stream, 1, A, R, S, gain, beta, Yn, rows, dim, eps, map);
    }
    return launched(add ? "residual_add_layer_norm" : "layer_norm");
}

elsa_status launch_act_inplace(uint16_t* Y, long long count, int act, elsa_dtype dtype, cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (count <= 0 || act == 0) return ELSA_OK;
    const long long vecs = count / 8;
    const unsigned grid = streaming_grid(vecs, 256, dev);
    ProfileScope scope(ELSA_KERNEL_BLOCK_ROWWISE, stream);
    if (dtype == ELSA_BF16) launch_pdl(act_inplace_kernel<true>, dim3(grid), dim3(256), 0, stream, 1, Y, vecs, act);
    else launch_pdl(act_inplace_kernel<false>, dim3(grid), dim3(256), 0, stream, 1, Y, vecs, act);
    return launched("act_inplace");
}

elsa_status launch_copy_columns(const uint16_t* src, uint16_t* dst, int rows, int src_ld, int col0, int cols,
                                cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (rows <= 0 || cols <= 0) return ELSA_OK;
    const unsigned grid = streaming_grid((long long)rows * (cols / 8), 256, dev);
    ProfileScope scope(ELSA_KERNEL_BLOCK_ROWWISE, stream);
    launch_pdl(copy_columns_kernel, dim3(grid), dim3(256), 0, stream, 1, src, dst, rows, src_ld, col0, cols);
    return launched("copy_columns");
}

}  // namespace elsa
