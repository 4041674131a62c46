// N:M sparse linear (N <= 2) on the 2:4 sparse MMA, on CTA pairs.
//
// Same product as elsa_sparse24.cu (Sec. 2, Fig. 2 bottom of the ELSA paper, on the 2-of-4
// re-encoding of the packed weight), organised so that the sparse MMA rate is not lost to operand
// traffic: the sparse rate doubles the bytes per cycle a tile needs, and a single CTA cannot stage
// them.  Two CTAs of a cluster share a tile of 256 features x 224 token rows: each CTA stages its
// own 128 compressed weight rows with their metadata and only half (112) of the activation rows,
// and the leader issues tcgen05.mma.sp.cta_group::2.  K advances in blocks of 128 (one 128-byte
// swizzle row of compressed weights, four metadata columns).  In the epilogue lanes are features:
// neighbouring lanes exchange one value per row pair so that every lane holds a feature pair, the
// 32 x 32 chunk is laid out row-major in swizzled shared memory with conflict-free 32-bit stores,
// and a TMA store writes it (and clips the ragged last rows).
//
// Per CTA (320 threads): warp 0 TMA producer, warp 1 tensor-memory allocation and (leader) MMA
// issue, warps 2-9 epilogue.  Waits are bounded as in the other tensor-core kernels.

#include <atomic>
#include <mutex>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kFeatPerCta = 128;   // compressed weight rows per CTA = TMEM lanes
constexpr int kPairFeat = 256;     // MMA M over the pair
constexpr int kRowTile = 224;      // token rows per pair tile = MMA N
constexpr int kRowsPerCta = kRowTile / 2;   // activation rows each CTA stages
constexpr int kBlockK = 128;       // logical K per stage
constexpr int kSpUmmaK = 32;
constexpr int kNumAccum = 2;
constexpr int kAccStride = 256;
constexpr int kMetaCol0 = kRowTile;   // 4 metadata columns per stage in [224, 256)
constexpr int kTmemCols = 512;
constexpr int kMaxStages = 8;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kEpiCols = 32;
constexpr int kATileBytes = kFeatPerCta * (kBlockK / 2) * 2;   // 16 KB: 128 rows of 128 bytes
constexpr int kBSubBytes = kRowsPerCta * 64 * 2;               // 14 KB: 112 rows of 128 bytes (64 k)
constexpr int kBTileBytes = 2 * kBSubBytes;                    // two 64-k halves
constexpr int kMetaBytes = 128 * 16;
constexpr int kStageBytes = kATileBytes + kBTileBytes + kMetaBytes;
constexpr int kStagingBytes = 32 * kEpiCols * 2;               // per warp, per buffer
constexpr int kStagingTotal = kEpiWarps * 2 * kStagingBytes;
constexpr int kBarrierBytes = 256;

static_assert(kStageBytes % 1024 == 0 && kBSubBytes % 1024 == 0, "swizzled tiles stay 1024-byte aligned");

// One layer of a launch; a launch may carry several (their tiles form one sequence, so one layer's
// tail overlaps the next one's head).  Lives in kernel-parameter space.
struct alignas(64) SpPairLayer {
    CUtensorMap map_a, map_x, map_e, map_y;
    int rows, out;
    int tiles_f;       // ceil(out / 256)
    int tile_begin;    // index of this layer's first tile in the launch's sequence
    int num_k_blocks;  // ceil(in / 128)
    const uint16_t* bias;
};

template <int kMaxLayers>
struct SpPairGroup {
    SpPairLayer layer[kMaxLayers];
    int n_layers;
    int num_tiles;
    int stages;
    uint32_t idesc;
    uint32_t* dev_status;
};

constexpr int kGroupMax = 56;   // layers per grouped launch (kernel parameters are limited to 32 KB)

template <bool kBf16, int kMaxLayers>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_sp24_pair_kernel(const __grid_constant__ SpPairGroup<kMaxLayers> p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    const uint32_t staging_base = smem_base + (uint32_t)(p.stages * kStageBytes);
    const uint32_t bar_off = (uint32_t)(p.stages * kStageBytes) + kStagingTotal;
    const uint32_t bar_base = smem_base + bar_off;
    const uint32_t full_bar = bar_base;                       // leader only
    const uint32_t empty_bar = bar_base + 8 * kMaxStages;     // per CTA
    const uint32_t tmem_full_bar = bar_base + 16 * kMaxStages;        // per CTA
    const uint32_t tmem_empty_bar = tmem_full_bar + 8 * kNumAccum;    // leader only
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
            mbar_init(tmem_empty_bar + 8 * a, 2 * kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc_pair(smem_base + holder_off, kTmemCols);
    tc_fence_before();
    __syncthreads();
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait_for_predecessors();
    pdl_release_successors();

    if (warp == 0) {
        // ------------------------------------------------ producer (both CTAs)
        // whole warp converged, one elected lane issues (see the MMA warp)
        {
            const bool elected = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int cur = 0;
            for (int tile = pair; ok && tile < p.num_tiles; tile += num_pairs) {
                while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
                const SpPairLayer& L = p.layer[cur];
                const int t = tile - L.tile_begin;
                const int ft128 = (t % L.tiles_f) * 2 + (int)cta_rank;   // this CTA's block of 128 features
                const int r0 = (t / L.tiles_f) * kRowTile + (int)cta_rank * kRowsPerCta;
                for (int kb = 0; kb < L.num_k_blocks; ++kb) {
                    ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    const uint32_t a_dst = smem_base + (uint32_t)(stage * kStageBytes);
                    const uint32_t bar = mapa_shared(full_bar + 8 * stage, 0);
                    if (elected) {
                        if (cta_rank == 0) mbar_arrive_expect_tx(full_bar + 8 * stage, (uint32_t)(2 * kStageBytes));
                        tma_load_2d_pair(a_dst, &L.map_a, bar, kb * (kBlockK / 2), ft128 * kFeatPerCta);
                        tma_load_2d_pair(a_dst + kATileBytes, &L.map_x, bar, kb * kBlockK, r0);
                        tma_load_2d_pair(a_dst + kATileBytes + kBSubBytes, &L.map_x, bar, kb * kBlockK + 64, r0);
                        tma_load_2d_pair(a_dst + kATileBytes + kBTileBytes, &L.map_e, bar, 0,
                                         (ft128 * L.num_k_blocks + kb) * 128);
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop with its operands in uniform registers; only the tensor-core
        // instructions are predicated on one elected lane (a single thread inside a divergent branch
        // needs about twice as long per MMA).
        if (cta_rank == 0) {
            const uint32_t elected = elect_one() ? 1u : 0u;
            // the base address came from shared memory in an ordinary register; a warp reduction returns it
            // in a uniform one, so that the addresses derived from it stay uniform too
            const uint32_t tmem_u = __reduce_or_sync(0xFFFFFFFFu, tmem_base);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            int cur = 0;
            for (int tile = pair; ok && tile < p.num_tiles; tile += num_pairs) {
                while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
                const int num_k_blocks = p.layer[cur].num_k_blocks;
                ok = mbar_wait(tmem_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_u + (uint32_t)(acc * kAccStride);
                for (int kb = 0; kb < num_k_blocks; ++kb) {
                    ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + (uint32_t)(stage * kStageBytes);
                    const uint64_t a_desc = smem_desc_k_major_sw128(a_addr);
                    const uint64_t b_desc0 = smem_desc_k_major_sw128(a_addr + kATileBytes);
                    const uint64_t b_desc1 = smem_desc_k_major_sw128(a_addr + kATileBytes + kBSubBytes);
                    const uint32_t e_col = tmem_u + (uint32_t)(kMetaCol0 + 4 * stage);
                    // each CTA's metadata block into its own tensor memory; runs before the MMAs below
                    const uint64_t e_desc = smem_desc_rows16_no_swizzle(a_addr + kATileBytes + kBTileBytes);
                    tmem_cp_128x128b_pair_if(e_col, e_desc, elected);
#pragma unroll
                    for (int j = 0; j < kBlockK / kSpUmmaK; ++j) {
                        // K step of 32: 32 bytes of compressed A, 64 bytes of B in the half that holds it
                        const uint64_t b_desc = (j < 2 ? b_desc0 : b_desc1) + (uint64_t)(4 * (j & 1));
                        umma_sp_f16_pair_if(d_tmem, a_desc + (uint64_t)(2 * j), b_desc, e_col + (uint32_t)j, p.idesc,
                                            (uint32_t)((kb | j) != 0), elected);
                    }
                    umma_commit_pair_if(empty_bar + 8 * stage, 3, elected);
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair_if(tmem_full_bar + 8 * acc, 3, elected);
                if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: lanes are features, columns are token rows
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;       // the two warps of a lane quarter take alternate chunks
        const uint32_t empty_remote = mapa_shared(tmem_empty_bar, 0);
        int acc = 0;
        uint32_t acc_phase = 0;
        constexpr int kChunks = kRowTile / kEpiCols;     // 7
        const int my_chunks = (kChunks - half + 1) / 2;  // 4 or 3
        const bool odd = (lane & 1) != 0;
        const uint32_t stage_buf = staging_base + (uint32_t)((warp - 2) * 2 * kStagingBytes);
        uint32_t chunk_counter = 0;
        // staging address pieces that do not depend on the row pair: the odd lane's row is one further
        // (64 bytes), the word inside the 16-byte chunk is (lane / 2) % 4, and the chunk index lane / 8
        // is xor-ed with (row / 2) % 4, one of four values
        const uint32_t prmt_sel = odd ? 0x7632u : 0x5410u;
        const uint32_t lane_off = (odd ? 64u : 0u) + (uint32_t)(((lane >> 1) & 3) * 4);
        uint32_t sw_off[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) sw_off[k] = (((uint32_t)(lane >> 3)) ^ (uint32_t)k) << 4;

        int cur = 0;
        for (int tile = pair; tile < p.num_tiles; tile += num_pairs) {
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            const SpPairLayer& L = p.layer[cur];
            const int t = tile - L.tile_begin;
            const int f0 = ((t % L.tiles_f) * 2 + (int)cta_rank) * kFeatPerCta + q * 32;
            const int r0 = (t / L.tiles_f) * kRowTile;
            const int f = f0 + lane;
            const int l_rows = L.rows, l_out = L.out;
            const uint16_t* l_bias = L.bias;
            const float bias_f = (l_bias != nullptr && f < l_out) ? bias_to_float<kBf16>(l_bias[f]) : 0.f;
            bool ok = mbar_wait(tmem_full_bar + 8 * acc, acc_phase, abort_flag, p.dev_status, 4);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kAccStride);
            auto emit = [&](const uint32_t (&r)[32], int c) {
                const uint32_t buf = stage_buf + (chunk_counter & 1u) * kStagingBytes;
                if (lane == 0) bulk_wait_group_read<1>();   // the store two chunks ago has drained this buffer
                __syncwarp();
                // staging tile [32 token rows][32 features], 64-byte rows with the 64-byte swizzle; this lane
                // writes the feature pair (lane & ~1, lane | 1) of one row per row pair
                // (all exchanges first, then all stores: interleaved, each store would wait for its shuffle)
                uint32_t word[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    // own feature, token rows j (low half) and j + 1 (high half), rounded once
                    const uint32_t own = pack2<kBf16>(__uint_as_float(r[j]) + bias_f, __uint_as_float(r[j + 1]) + bias_f);
                    const uint32_t got = __shfl_xor_sync(0xFFFFFFFFu, own, 1);
                    // even lane: row j of (own, right neighbour); odd lane: row j + 1 of (left neighbour, own)
                    asm("prmt.b32 %0, %1, %2, %3;" : "=r"(word[j >> 1]) : "r"(odd ? got : own), "r"(odd ? own : got), "r"(prmt_sel));
                }
#pragma unroll
                for (int j = 0; j < 32; j += 2)
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(buf + lane_off + (uint32_t)(j * 64) + sw_off[(j >> 1) & 3]),
                                 "r"(word[j >> 1])
                                 : "memory");
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int row0 = r0 + c * kEpiCols;
                    if (row0 < l_rows && f0 < l_out) tma_store_2d(&L.map_y, buf, f0, row0);
                    bulk_commit_group();
                }
                ++chunk_counter;
            };
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(empty_remote + 8 * acc);
            };

            uint32_t ra[32], rb[32];
            tmem_ld_32x32b_x32(t_row + (uint32_t)(half * kEpiCols), ra);
            for (int i = 0; i < my_chunks; i += 2) {
                tmem_wait_ld();
                if (i + 1 < my_chunks) tmem_ld_32x32b_x32(t_row + (uint32_t)((half + 2 * (i + 1)) * kEpiCols), rb);
                else release();
                emit(ra, half + 2 * i);
                if (i + 1 < my_chunks) {
                    tmem_wait_ld();
                    if (i + 2 < my_chunks) tmem_ld_32x32b_x32(t_row + (uint32_t)((half + 2 * (i + 2)) * kEpiCols), ra);
                    else release();
                    emit(rb, half + 2 * (i + 1));
                }
            }
            if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_group_all();
        __syncwarp();
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        for (int i = 0; i < 200; ++i) __nanosleep(10000);
    }
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

}  // namespace

namespace {

template <bool kBf16, int kMaxLayers>
elsa_status launch_sp_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status, cudaStream_t stream,
                            const DeviceInfo& dev)
{
    static SpPairGroup<kMaxLayers> g;   // host staging of the kernel parameters
    static std::mutex g_mutex;
    std::lock_guard<std::mutex> lock(g_mutex);
    int tile_begin = 0;
    for (int i = 0; i < n; ++i) {
        const SparseJob& j = jobs[i];
        SpPairLayer& L = g.layer[i];
        const int tiles_f128 = (j.out + kFeatPerCta - 1) / kFeatPerCta;
        L.rows = j.rows; L.out = j.out;
        L.tiles_f = (j.out + kPairFeat - 1) / kPairFeat;
        L.tile_begin = tile_begin;
        tile_begin += L.tiles_f * ((j.rows + kRowTile - 1) / kRowTile);
        L.num_k_blocks = (j.in + kBlockK - 1) / kBlockK;
        L.bias = j.bias;
        const uint16_t* a_img = (const uint16_t*)j.workspace;
        const uint8_t* meta = (const uint8_t*)j.workspace + sp24_meta_offset(j.out, j.in);
        elsa_status st;
        if ((st = make_map_2d(&L.map_a, a_img, (uint64_t)(j.in / 2), (uint64_t)j.out, kBlockK / 2, kFeatPerCta,
                              CU_TENSOR_MAP_SWIZZLE_128B, "2:4 weight image")) != ELSA_OK)
            return st;
        if ((st = make_map_2d(&L.map_x, j.X, (uint64_t)j.in, (uint64_t)j.rows, 64, kRowsPerCta, CU_TENSOR_MAP_SWIZZLE_128B,
                              "X")) != ELSA_OK)
            return st;
        // metadata blocks as a matrix of 16-byte rows: 128 rows per (128 features, K block)
        if ((st = make_map_2d(&L.map_e, meta, 8, (uint64_t)tiles_f128 * L.num_k_blocks * 128, 8, 128,
                              CU_TENSOR_MAP_SWIZZLE_NONE, "metadata")) != ELSA_OK)
            return st;
        if ((st = make_map_2d(&L.map_y, j.Y, (uint64_t)j.out, (uint64_t)j.rows, kEpiCols, 32, CU_TENSOR_MAP_SWIZZLE_64B,
                              "Y")) != ELSA_OK)
            return st;
    }
    g.n_layers = n;
    g.num_tiles = tile_begin;
    g.dev_status = dev_status;
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    // sparse flag, fp32 accumulate, A and B of type fmt, K-major, N = 224, M = 256 over the pair
    g.idesc = (1u << 2) | (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRowTile >> 3) << 17) |
              ((uint32_t)(kPairFeat >> 4) << 24);

    const int fixed = kStagingTotal + kBarrierBytes + 1024;
    int stages = (int)((dev.smem_optin - fixed) / kStageBytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(ELSA_ERR_CUDA, "not enough shared memory for two pipeline stages");
    g.stages = stages;
    const size_t smem = (size_t)stages * kStageBytes + fixed;

    auto kernel = linear_tc_sp24_pair_kernel<kBf16, kMaxLayers>;
    static std::atomic<int> max_pairs[64];   // zero-initialised; racing first calls compute the same value
    const int slot = dev.device & 63;
    if (max_pairs[slot].load(std::memory_order_acquire) == 0) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dev.smem_optin) !=
            cudaSuccess) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        cudaLaunchConfig_t cfg = {};
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.gridDim = dim3((unsigned)dev.sm_count);
        cfg.blockDim = dim3(kThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int m = 0;
        if (cudaOccupancyMaxActiveClusters(&m, kernel, &cfg) != cudaSuccess || m < 1) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaOccupancyMaxActiveClusters: %s", cudaGetErrorString(e));
        }
        max_pairs[slot].store(m, std::memory_order_release);
    }
    const int pairs = g.num_tiles < max_pairs[slot].load(std::memory_order_acquire) ? g.num_tiles : max_pairs[slot].load(std::memory_order_acquire);
    ProfileScope scope(ELSA_KERNEL_LINEAR_TC_SP24_PAIR, stream);
    cudaError_t e = launch_pdl(kernel, dim3((unsigned)(2 * pairs)), dim3(kThreads), smem, stream, 2, g);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ELSA_ERR_CUDA, "launch of linear_tc_sp24_pair failed: %s", cudaGetErrorString(e));
    }
    return launched("linear_tc_sp24_pair");
}

}  // namespace

int linear_tc_sparse_pair_group_max() { return kGroupMax; }

elsa_status launch_linear_tc_sparse_pair_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                               cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (n < 1 || n > kGroupMax) return fail(ELSA_ERR_SHAPE, "a grouped launch carries 1 to %d layers, got %d", kGroupMax, n);
    if (n == 1)
        return dtype == ELSA_BF16 ? launch_sp_group<true, 1>(jobs, 1, dtype, dev_status, stream, dev)
                                  : launch_sp_group<false, 1>(jobs, 1, dtype, dev_status, stream, dev);
    return dtype == ELSA_BF16 ? launch_sp_group<true, kGroupMax>(jobs, n, dtype, dev_status, stream, dev)
                              : launch_sp_group<false, kGroupMax>(jobs, n, dtype, dev_status, stream, dev);
}

elsa_status launch_linear_tc_sparse_pair(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                         const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype,
                                         uint16_t* Y, void* workspace, uint32_t* dev_status, cudaStream_t stream)
{
    if (!linear_tc_sparse_suits(in, N) || N == M)
        return fail(ELSA_ERR_NM, "level %d:%d with in=%d does not fit the 2:4 sparse MMA path", N, M, in);
    elsa_status st = launch_linear_tc_sparse_pair_prepare(vals, idx, out, in, N, M, SP24_ROWS, workspace, stream);
    if (st != ELSA_OK) return st;
    SparseJob job;
    job.X = X; job.bias = bias; job.Y = Y; job.workspace = workspace;
    job.rows = rows; job.in = in; job.out = out;
    return launch_linear_tc_sparse_pair_group(&job, 1, dtype, dev_status, stream);
}

// Re-encodes one packed weight into `workspace` in the form the pair kernel reads (K blocks of 128).
elsa_status launch_linear_tc_sparse_pair_prepare(const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                                                 int layout, void* workspace, cudaStream_t stream)
{
    uint16_t* a_img = (uint16_t*)workspace;
    uint8_t* meta = (uint8_t*)workspace + sp24_meta_offset(out, in);
    return launch_nm_to_sp24(vals, idx, out, in, N, M, kBlockK, layout, a_img, meta, stream);
}

}  // namespace elsa
