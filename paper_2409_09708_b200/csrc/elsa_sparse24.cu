// N:M sparse linear on the hardware 2:4 sparse MMA of sm_100a, for levels with N <= 2.
//
// Sec. 2, Fig. 2 bottom of the ELSA paper: the index of each kept weight selects the activation it
// multiplies, and only kept weights are multiplied.  The tensor cores offer exactly one form of
// that: tcgen05.mma.sp, whose A operand holds 2 values out of every aligned chunk of 4 along K,
// with 2-bit positions as metadata.  Every N:M pattern with N <= 2 (1:4, 2:4, 1:8, 2:8, 1:16,
// 2:16) has at most 2 kept weights in each aligned 4-chunk, so the packed weight can be
// re-encoded, without loss, as 2-of-4 (zero padded) and run at the sparse MMA rate: half of the
// multiply-accumulates of the dense image are never issued.
//
// Two kernels:
//   nm_to_sp24_kernel   packed (vals, idx) -> A image [out][in/2] (2 values per 4-chunk, in
//                       ascending position) + metadata blocks laid out as tensor memory wants them
//   linear_tc_sp24_kernel   persistent tcgen05 GEMM with the sparse operand on the M side:
//                       D[feature lanes][token columns] = Wsp[128 x K] * X[BN x K]^T, so the epilogue
//                       transposes through shared memory on its way to row-major Y.
//
// Metadata in tensor memory (16-bit types): one 32-bit column per K step of 32; lane
// L = (m % 8) + 8 * ((k / 16) % 2) + 16 * (m / 16) holds, in its low half-word, the four nibbles of
// row m (with (m / 8) % 2 == 0) for the 16 k of that half step, and in its high half-word those of
// row m + 8; nibble c of a half-word describes chunk c: position of the first stored value in bits
// 0-1, of the second in bits 2-3 (first < second).

#include "elsa_pack_device.cuh"
#include <atomic>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kFeatTile = 128;     // features per tile = MMA M = TMEM lanes
constexpr int kRowTile = 224;      // token rows per tile = MMA N (leaves 32 TMEM columns per half for metadata)
constexpr int kBlockK = 64;        // logical K per stage
constexpr int kSpUmmaK = 32;       // logical K per sparse MMA for 16-bit inputs
constexpr int kNumAccum = 2;
constexpr int kAccStride = 256;    // TMEM columns between the two accumulators
constexpr int kMetaCol0 = kRowTile;  // metadata ring: 4 columns per stage in [224, 256)
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 8;
constexpr int kEpiWarps = 4;
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kEpiCols = 32;
constexpr int kATileBytes = kFeatTile * (kBlockK / 2) * 2;   // 8 KB: 128 rows of 64 bytes
constexpr int kBTileBytes = kRowTile * kBlockK * 2;          // 28 KB: 224 rows of 128 bytes
constexpr int kMetaBytes = 128 * 16;                         // 2 KB: 16 bytes per lane, 8 of them used
constexpr int kStageBytes = kATileBytes + kBTileBytes + kMetaBytes;
constexpr int kStagingBytes = 32 * kEpiCols * 2;
constexpr int kStagingTotal = kEpiWarps * 2 * kStagingBytes;
constexpr int kBarrierBytes = 256;

static_assert(kStageBytes % 1024 == 0, "stages keep the 1024-byte alignment of the swizzled tiles");

// ------------------------------------------------------------------ re-encoding

// (the per-segment device code is in elsa_pack_device.cuh)
template <int M>
__global__ void __launch_bounds__(256)
nm_to_sp24_kernel(const uint16_t* __restrict__ vals, const uint32_t* __restrict__ idx, int out, int in, int N,
                  int words_per_row, uint16_t* __restrict__ a_img, uint16_t* __restrict__ meta16, int out_tiles,
                  int k_blocks, int steps_per_block, int layout)
{
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (tid >= (long long)out_tiles * kFeatTile * k_blocks * steps_per_block * 2) return;
    to_sp24_segment<M>(vals, idx, out, in, N, words_per_row, a_img, meta16, k_blocks, steps_per_block, layout, tid);
}

template <int M>
__global__ void __launch_bounds__(256)
dense_to_sp24_kernel(const uint16_t* __restrict__ W, int out, int in, int N, uint16_t* __restrict__ a_img,
                     uint16_t* __restrict__ meta16, int out_tiles, int k_blocks, int steps_per_block, int layout)
{
    const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (tid >= (long long)out_tiles * kFeatTile * k_blocks * steps_per_block * 2) return;
    dense_to_sp24_segment<M>(W, out, in, N, a_img, meta16, k_blocks, steps_per_block, layout, tid);
}

// ------------------------------------------------------------------ GEMM

struct SpParams {
    int rows, in, out;
    int tiles_f;       // ceil(out / 128)
    int num_tiles;
    int num_k_blocks;
    int stages;
    uint32_t idesc;
    const uint16_t* bias;
    const uint8_t* meta;   // metadata blocks
    uint32_t* dev_status;
};

template <bool kBf16>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_sp24_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_x,
                      const __grid_constant__ CUtensorMap map_y, const SpParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    const uint32_t staging_base = smem_base + (uint32_t)(p.stages * kStageBytes);
    const uint32_t bar_off = (uint32_t)(p.stages * kStageBytes) + kStagingTotal;
    const uint32_t bar_base = smem_base + bar_off;
    const uint32_t full_bar = bar_base;
    const uint32_t empty_bar = bar_base + 8 * kMaxStages;
    const uint32_t tmem_full_bar = bar_base + 16 * kMaxStages;
    const uint32_t tmem_empty_bar = tmem_full_bar + 8 * kNumAccum;
    const uint32_t holder_off = bar_off + 16 * kMaxStages + 16 * kNumAccum;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < kNumAccum; ++a) {
            mbar_init(tmem_full_bar + 8 * a, 1);
            mbar_init(tmem_empty_bar + 8 * a, kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc(smem_base + holder_off, kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait_for_predecessors();
    pdl_release_successors();

    if (warp == 0) {
        // ------------------------------------------------ producer: W (2:4 image), X and metadata per K block
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
                const int ft = tile % p.tiles_f;                  // feature tiles fastest: CTAs share X in L2
                const int r0 = (tile / p.tiles_f) * kRowTile;
                for (int kb = 0; kb < p.num_k_blocks; ++kb) {
                    ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                    if (!ok) break;
                    const uint32_t a_dst = smem_base + (uint32_t)(stage * kStageBytes);
                    const uint32_t bar = full_bar + 8 * stage;
                    mbar_arrive_expect_tx(bar, (uint32_t)kStageBytes);
                    tma_load_2d(a_dst, &map_a, bar, kb * (kBlockK / 2), ft * kFeatTile);
                    tma_load_2d(a_dst + kATileBytes, &map_x, bar, kb * kBlockK, r0);
                    bulk_load_1d(a_dst + kATileBytes + kBTileBytes,
                                 p.meta + ((size_t)ft * p.num_k_blocks + kb) * kMetaBytes, kMetaBytes, bar);
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
                ok = mbar_wait(tmem_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kAccStride);
                for (int kb = 0; kb < p.num_k_blocks; ++kb) {
                    ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + (uint32_t)(stage * kStageBytes);
                    const uint64_t a_desc = smem_desc_k_major_sw64(a_addr);
                    const uint64_t b_desc = smem_desc_k_major_sw128(a_addr + kATileBytes);
                    const uint32_t e_col = tmem_base + (uint32_t)(kMetaCol0 + 4 * stage);
                    // metadata of this K block into its 4 ring columns; executes before the MMAs below
                    tmem_cp_128x128b(e_col, smem_desc_rows16_no_swizzle(a_addr + kATileBytes + kBTileBytes));
#pragma unroll
                    for (int j = 0; j < kBlockK / kSpUmmaK; ++j) {
                        // one K step of 32: 16 stored A elements (32 bytes), 32 B elements (64 bytes)
                        umma_sp_f16(d_tmem, a_desc + (uint64_t)(2 * j), b_desc + (uint64_t)(4 * j), e_col + (uint32_t)j,
                                    p.idesc, (uint32_t)((kb | j) != 0));
                    }
                    umma_commit(empty_bar + 8 * stage);
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit(tmem_full_bar + 8 * acc);
                if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: lanes are features, columns are token rows
        const int q = warp & 3;
        const int ew = warp - 2;
        const uint32_t stage_buf = staging_base + (uint32_t)(ew * 2 * kStagingBytes);
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t chunk_counter = 0;
        constexpr int kChunks = kRowTile / kEpiCols;
        for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
            const int f0 = (tile % p.tiles_f) * kFeatTile + q * 32;     // first feature of this warp
            const int r0 = (tile / p.tiles_f) * kRowTile;
            const int f = f0 + lane;
            const float bias_f = (p.bias != nullptr && f < p.out) ? bias_to_float<kBf16>(p.bias[f]) : 0.f;
            bool ok = mbar_wait(tmem_full_bar + 8 * acc, acc_phase, abort_flag, p.dev_status, 4);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccStride);
            for (int c = 0; c < kChunks; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(t_row + (uint32_t)(c * kEpiCols), r);
                tmem_wait_ld();
                if (c == kChunks - 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tmem_empty_bar + 8 * acc);
                }
                const uint32_t buf = stage_buf + (chunk_counter & 1u) * kStagingBytes;
                if (lane == 0) bulk_wait_group_read<1>();
                __syncwarp();
                // staging tile [32 token rows][32 features], rows of 64 bytes with the 64-byte swizzle;
                // this thread owns feature column `lane`: 16-byte chunk lane / 8, 2-byte slot lane % 8
                const uint32_t col_chunk = (uint32_t)(lane >> 3);
                const uint32_t col_off = (uint32_t)((lane & 7) * 2);
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const float v = __uint_as_float(r[j]) + bias_f;
                    uint16_t h;
                    if constexpr (kBf16) h = __bfloat16_as_ushort(__float2bfloat16_rn(v));
                    else h = __half_as_ushort(__float2half_rn(v));
                    const uint32_t addr = buf + (uint32_t)(j * 64) + ((col_chunk ^ (uint32_t)((j >> 1) & 3)) << 4) + col_off;
                    asm volatile("st.shared.u16 [%0], %1;" ::"r"(addr), "h"(h) : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int row0 = r0 + c * kEpiCols;
                    if (row0 < p.rows && f0 < p.out) tma_store_2d(&map_y, buf, f0, row0);
                    bulk_commit_group();
                }
                ++chunk_counter;
            }
            if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_group_all();
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) {
            for (int i = 0; i < 200; ++i) __nanosleep(10000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

elsa_status launch_nm_to_sp24(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M, int block_k,
                              int layout, uint16_t* a_img, uint8_t* meta, cudaStream_t stream)
{
    const int perm = layout;
    const int tiles_f = (out + kFeatTile - 1) / kFeatTile;
    const int k_blocks = (in + block_k - 1) / block_k;
    const int steps = block_k / kSpUmmaK;
    const long long threads = (long long)tiles_f * kFeatTile * k_blocks * steps * 2;
    const unsigned grid = (unsigned)((threads + 255) / 256);
    const int wpr = (int)index_words_per_row(in, N, M);
    ProfileScope scope(ELSA_KERNEL_NM_TO_SP24, stream);
    if (M == 4)
        launch_pdl(nm_to_sp24_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, wpr, a_img,
                   (uint16_t*)meta, tiles_f, k_blocks, steps, perm);
    else if (M == 8)
        launch_pdl(nm_to_sp24_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, wpr, a_img,
                   (uint16_t*)meta, tiles_f, k_blocks, steps, perm);
    else
        launch_pdl(nm_to_sp24_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, vals, idx, out, in, N, wpr, a_img,
                   (uint16_t*)meta, tiles_f, k_blocks, steps, perm);
    return launched("nm_to_sp24");
}

elsa_status launch_dense_to_sp24(const uint16_t* W, int out, int in, int N, int M, int block_k, int layout,
                                 uint16_t* a_img, uint8_t* meta, cudaStream_t stream)
{
    const int perm = layout;
    const int tiles_f = (out + kFeatTile - 1) / kFeatTile;
    const int k_blocks = (in + block_k - 1) / block_k;
    const int steps = block_k / kSpUmmaK;
    const long long threads = (long long)tiles_f * kFeatTile * k_blocks * steps * 2;
    const unsigned grid = (unsigned)((threads + 255) / 256);
    ProfileScope scope(ELSA_KERNEL_NM_TO_SP24, stream);
    if (M == 4)
        launch_pdl(dense_to_sp24_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, W, out, in, N, a_img, (uint16_t*)meta,
                   tiles_f, k_blocks, steps, perm);
    else if (M == 8)
        launch_pdl(dense_to_sp24_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, W, out, in, N, a_img, (uint16_t*)meta,
                   tiles_f, k_blocks, steps, perm);
    else
        launch_pdl(dense_to_sp24_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, W, out, in, N, a_img, (uint16_t*)meta,
                   tiles_f, k_blocks, steps, perm);
    return launched("dense_to_sp24");
}

bool linear_tc_sparse_suits(int in, int N)
{
    // the 2:4 image needs at most 2 kept weights per aligned 4-chunk (guaranteed for N <= 2) and
    // whole 16-k segments with a 16-byte row pitch of the half-width image
    return N <= 2 && in % 16 == 0;
}

size_t linear_tc_sparse_workspace(int out, int in)
{
    const size_t tiles = (size_t)(out + kFeatTile - 1) / kFeatTile;
    const size_t kbs = (size_t)(in + kBlockK - 1) / kBlockK;
    return sp24_meta_offset(out, in) + tiles * kbs * kMetaBytes;
}

elsa_status launch_linear_tc_sparse(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                    const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype, uint16_t* Y,
                                    void* workspace, uint32_t* dev_status, cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (!linear_tc_sparse_suits(in, N) || N == M)
        return fail(ELSA_ERR_NM, "level %d:%d with in=%d does not fit the 2:4 sparse MMA path", N, M, in);

    const int tiles_f = (out + kFeatTile - 1) / kFeatTile;
    const int k_blocks = (in + kBlockK - 1) / kBlockK;
    uint16_t* a_img = (uint16_t*)workspace;
    uint8_t* meta = (uint8_t*)workspace + sp24_meta_offset(out, in);

    if ((st = launch_nm_to_sp24(vals, idx, out, in, N, M, kBlockK, SP24_ROWS, a_img, meta, stream)) != ELSA_OK) return st;

    SpParams p;
    p.rows = rows; p.in = in; p.out = out;
    p.tiles_f = tiles_f;
    p.num_tiles = tiles_f * ((rows + kRowTile - 1) / kRowTile);
    p.num_k_blocks = k_blocks;
    p.bias = bias;
    p.meta = meta;
    p.dev_status = dev_status;
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    // sparse flag (bit 2), fp32 accumulate, A and B of type fmt, K-major, N = 224, M = 128
    p.idesc = (1u << 2) | (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRowTile >> 3) << 17) |
              ((uint32_t)(kFeatTile >> 4) << 24);

    const int fixed = kStagingTotal + kBarrierBytes + 1024;
    int stages = (int)((dev.smem_optin - fixed) / kStageBytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(ELSA_ERR_CUDA, "not enough shared memory for two pipeline stages");
    p.stages = stages;
    const size_t smem = (size_t)stages * kStageBytes + fixed;

    CUtensorMap map_a, map_x, map_y;
    if ((st = make_map_2d(&map_a, a_img, (uint64_t)(in / 2), (uint64_t)out, kBlockK / 2, kFeatTile,
                          CU_TENSOR_MAP_SWIZZLE_64B, "2:4 weight image")) != ELSA_OK)
        return st;
    if ((st = make_map_2d(&map_x, X, (uint64_t)in, (uint64_t)rows, kBlockK, kRowTile, CU_TENSOR_MAP_SWIZZLE_128B, "X")) !=
        ELSA_OK)
        return st;
    if ((st = make_map_2d(&map_y, Y, (uint64_t)out, (uint64_t)rows, kEpiCols, 32, CU_TENSOR_MAP_SWIZZLE_64B, "Y")) !=
        ELSA_OK)
        return st;

    static std::atomic<bool> attr_set[64][2];   // zero-initialised; a double set by racing threads is harmless
    auto kernel = dtype == ELSA_BF16 ? linear_tc_sp24_kernel<true> : linear_tc_sp24_kernel<false>;
    const int slot = dev.device & 63;
    if (!attr_set[slot][fmt].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dev.smem_optin) !=
            cudaSuccess) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        attr_set[slot][fmt].store(true, std::memory_order_release);
    }
    const int grid = p.num_tiles < dev.sm_count ? p.num_tiles : dev.sm_count;
    ProfileScope scope(ELSA_KERNEL_LINEAR_TC_SP24, stream);
    launch_pdl(kernel, dim3(grid), dim3(kThreads), smem, stream, 1, map_a, map_x, map_y, p);
    return launched("linear_tc_sp24");
}

}  // namespace elsa
