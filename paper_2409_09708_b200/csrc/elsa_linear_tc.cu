// Tensor-core linear for sm_100a: Y[rows][out] = X[rows][in] * Wd[out][in]^T + bias.
//
// This is the contraction step of the N:M sparse product (Sec. 2, Fig. 2 bottom of the ELSA paper):
// once a weight tile has been put back at its positions it is a dense contraction, so it runs
// on the 5th-generation tensor cores.  Wd is the weight as the MMA reads it: either the dense
// level's values themselves (N == M) or the image the expand kernel rebuilt from the packed form.
//
// Structure (one persistent CTA per SM, 192 threads):
//   warp 0      TMA producer: X tile [128 x 64] and W tile [BN x 64] per K block into a ring of
//               shared-memory stages (128-byte swizzle), signalled through mbarriers
//   warp 1      allocates tensor memory; one lane issues tcgen05.mma (M = 128, N = BN, K = 16) into
//               one of two TMEM accumulators and commits stage / accumulator barriers
//   warps 2-5   epilogue: tcgen05.ld the finished accumulator, add bias in fp32, round to 16 bit,
//               stage through swizzled shared memory and write Y with TMA stores (which clip the
//               ragged last row tile); overlaps the next tile's MMAs
// Tiles are visited feature-fastest so that the CTAs running together share X row blocks in L2.
// Every wait is bounded: on expiry the kernel records ELSA_ERR_TIMEOUT and all roles leave.

#include <atomic>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kBlockM = 128;       // token rows per tile = MMA M = TMEM lanes
constexpr int kBlockK = 64;        // one 128-byte swizzle row of 16-bit elements
constexpr int kUmmaK = 16;         // K per tcgen05.mma for 16-bit inputs
constexpr int kMaxBlockN = 256;    // features per tile = MMA N (<= 256)
constexpr int kNumAccum = 2;       // TMEM accumulators (MMA of tile i+1 overlaps epilogue of i)
constexpr int kTmemCols = kNumAccum * kMaxBlockN;
constexpr int kMaxStages = 8;
constexpr int kThreads = 192;
constexpr int kEpiWarps = 4;
constexpr int kEpiCols = 32;       // columns per epilogue chunk (one tcgen05.ld.32x32b.x32)
constexpr int kATileBytes = kBlockM * kBlockK * 2;
constexpr int kStagingBytes = 32 * kEpiCols * 2;             // per warp, per buffer
constexpr int kStagingTotal = kEpiWarps * 2 * kStagingBytes;
constexpr int kBiasBytes = kEpiWarps * kMaxBlockN * 4;
constexpr int kBarrierBytes = 256;

struct TcParams {
    int rows, in, out;
    int bn;            // features per tile
    int tiles_n;       // ceil(out / bn)
    int num_tiles;
    int num_k_blocks;  // ceil(in / 64)
    int stages;
    uint32_t idesc;
    const uint16_t* bias;
    uint32_t* dev_status;
};

// ------------------------------------------------------------------ kernel

template <bool kBf16>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_dense_kernel(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w,
                       const __grid_constant__ CUtensorMap map_y, const TcParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int b_tile_bytes = p.bn * kBlockK * 2;
    const int stage_bytes = kATileBytes + b_tile_bytes;

    const uint32_t staging_base = smem_base + (uint32_t)(p.stages * stage_bytes);
    const uint32_t bias_off = (uint32_t)(p.stages * stage_bytes) + kStagingTotal;
    const uint32_t bar_base = smem_base + bias_off + kBiasBytes;
    // barrier block: full[8], empty[8], tmem_full[2], tmem_empty[2], tmem holder, abort flag
    const uint32_t full_bar = bar_base;
    const uint32_t empty_bar = bar_base + 8 * kMaxStages;
    const uint32_t tmem_full_bar = bar_base + 16 * kMaxStages;
    const uint32_t tmem_empty_bar = tmem_full_bar + 8 * kNumAccum;
    const uint32_t holder_off = bias_off + kBiasBytes + 16 * kMaxStages + 16 * kNumAccum;
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
    // set-up above touched no global memory; from here on the predecessor's writes are needed
    pdl_wait_for_predecessors();
    pdl_release_successors();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        // whole warp converged, one elected lane issues (see the MMA warp)
        {
            const bool elected = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
                const int m0 = (tile / p.tiles_n) * kBlockM;
                const int n0 = (tile % p.tiles_n) * p.bn;
                for (int kb = 0; kb < p.num_k_blocks; ++kb) {
                    ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    const uint32_t a_dst = smem_base + (uint32_t)(stage * stage_bytes);
                    const uint32_t bar = full_bar + 8 * stage;
                    if (elected) {
                        mbar_arrive_expect_tx(bar, (uint32_t)stage_bytes);
                        tma_load_2d(a_dst, &map_x, bar, kb * kBlockK, m0);
                        tma_load_2d(a_dst + kATileBytes, &map_w, bar, kb * kBlockK, n0);
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer
        // The whole warp walks the loop with its operands in uniform registers; only the tensor-core
        // instructions are predicated on one elected lane (a single thread inside a divergent branch
        // needs about twice as long per MMA).
        {
            const uint32_t elected = elect_one() ? 1u : 0u;
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            bool ok = true;
            for (int tile = blockIdx.x; ok && tile < p.num_tiles; tile += gridDim.x) {
                ok = mbar_wait(tmem_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(acc * kMaxBlockN);
                for (int kb = 0; kb < p.num_k_blocks; ++kb) {
                    ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + (uint32_t)(stage * stage_bytes);
                    const uint64_t a_desc = smem_desc_k_major_sw128(a_addr);
                    const uint64_t b_desc = smem_desc_k_major_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        // advancing K by 16 elements = 32 bytes inside the swizzle row: +2 in the
                        // 16-byte-unit start address field
                        umma_f16_if(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), p.idesc,
                                    (uint32_t)((kb | k) != 0), elected);
                    }
                    umma_commit_if(empty_bar + 8 * stage, elected);  // frees the stage once these MMAs have read it
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_if(tmem_full_bar + 8 * acc, elected);    // accumulator complete
                if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue (warps 2..5)
        const int q = warp & 3;          // TMEM lane quarter this warp may read
        const int ew = warp - 2;         // private staging / bias slot
        const uint32_t stage_buf = staging_base + (uint32_t)(ew * 2 * kStagingBytes);
        float* bias_s = reinterpret_cast<float*>(smem_gen + bias_off) + ew * kMaxBlockN;
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t chunk_counter = 0;
        const int chunks = p.bn / kEpiCols;
        for (int tile = blockIdx.x; tile < p.num_tiles; tile += gridDim.x) {
            const int m0 = (tile / p.tiles_n) * kBlockM;
            const int n0 = (tile % p.tiles_n) * p.bn;
            for (int j = lane; j < p.bn; j += 32) {
                const int o = n0 + j;
                bias_s[j] = (p.bias != nullptr && o < p.out) ? bias_to_float<kBf16>(p.bias[o]) : 0.f;
            }
            __syncwarp();
            bool ok = mbar_wait(tmem_full_bar + 8 * acc, acc_phase, abort_flag, p.dev_status, 4);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kMaxBlockN);
            const int row0 = m0 + q * 32;
            for (int c = 0; c < chunks; ++c) {
                uint32_t r[32];
                tmem_ld_32x32b_x32(t_row + (uint32_t)(c * kEpiCols), r);
                tmem_wait_ld();
                if (c == chunks - 1) {
                    // accumulator fully read: hand it back to the MMA issuer
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tmem_empty_bar + 8 * acc);
                }
                uint32_t packed[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float2 b = *reinterpret_cast<const float2*>(bias_s + c * kEpiCols + 2 * j);
                    packed[j] = pack2<kBf16>(__uint_as_float(r[2 * j]) + b.x,
                                             __uint_as_float(r[2 * j + 1]) + b.y);
                }
                const uint32_t buf = stage_buf + (chunk_counter & 1u) * kStagingBytes;
                // the store that last read this buffer (two chunks ago) must have drained it
                if (lane == 0) bulk_wait_group_read<1>();
                __syncwarp();
                // staging rows are 64 bytes; 64-byte swizzle: 16-byte chunk index ^= (row / 2) % 4
                const uint32_t row_addr = buf + (uint32_t)(lane * 64);
                const uint32_t sw = (uint32_t)((lane >> 1) & 3);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(
                                     row_addr + (((uint32_t)j ^ sw) << 4)),
                                 "r"(packed[4 * j]), "r"(packed[4 * j + 1]), "r"(packed[4 * j + 2]),
                                 "r"(packed[4 * j + 3])
                                 : "memory");
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int col0 = n0 + c * kEpiCols;
                    if (row0 < p.rows && col0 < p.out) tma_store_2d(&map_y, buf, col0, row0);
                    bulk_commit_group();
                }
                ++chunk_counter;
            }
            if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_group_all();
        __syncwarp();
    }

    // ------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        if (*abort_flag) {
            // a wait gave up: let copies and MMAs that may still be in flight land before the
            // tensor memory and the shared memory are released
            for (int i = 0; i < 200; ++i) __nanosleep(10000);
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

int pick_block_n(int out, int tiles_m, int sm_count)
{
    // widest tile that wastes no more than one 64-feature slice, narrowed when the grid would
    // leave most SMs idle
    int best = 64, best_waste = 1 << 30;
    const int cand[4] = {256, 192, 128, 64};
    for (int i = 0; i < 4; ++i) {
        const int bn = cand[i];
        const int tiles_n = (out + bn - 1) / bn;
        const int waste = tiles_n * bn - out;
        if (waste < best_waste) { best = bn; best_waste = waste; }
    }
    while (best > 64 && tiles_m * ((out + best - 1) / best) < sm_count && best % 2 == 0 &&
           (best / 2) % 32 == 0)
        best /= 2;
    return best;
}

}  // namespace

elsa_status launch_linear_tc_dense(const uint16_t* X, int rows, const uint16_t* Wd, const uint16_t* bias,
                                   int out, int in, elsa_dtype dtype, uint16_t* Y, uint32_t* dev_status,
                                   cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;

    TcParams p;
    p.rows = rows; p.in = in; p.out = out;
    const int tiles_m = (rows + kBlockM - 1) / kBlockM;
    p.bn = pick_block_n(out, tiles_m, dev.sm_count);
    p.tiles_n = (out + p.bn - 1) / p.bn;
    p.num_tiles = tiles_m * p.tiles_n;
    p.num_k_blocks = (in + kBlockK - 1) / kBlockK;
    p.bias = bias;
    p.dev_status = dev_status;
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    // instruction descriptor: fp32 accumulate, A and B of type fmt, both K-major, N and M extents
    p.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(p.bn >> 3) << 17) |
              ((uint32_t)(kBlockM >> 4) << 24);

    const int stage_bytes = kATileBytes + p.bn * kBlockK * 2;
    const int fixed = kStagingTotal + kBiasBytes + kBarrierBytes + 1024;
    int stages = (int)((dev.smem_optin - fixed) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(ELSA_ERR_CUDA, "not enough shared memory for two pipeline stages");
    p.stages = stages;
    const size_t smem = (size_t)stages * stage_bytes + fixed;

    CUtensorMap map_x, map_w, map_y;
    if ((st = make_map_2d(&map_x, X, (uint64_t)in, (uint64_t)rows, kBlockK, kBlockM, CU_TENSOR_MAP_SWIZZLE_128B,
                          "X")) != ELSA_OK)
        return st;
    if ((st = make_map_2d(&map_w, Wd, (uint64_t)in, (uint64_t)out, kBlockK, (uint32_t)p.bn,
                          CU_TENSOR_MAP_SWIZZLE_128B, "W")) != ELSA_OK)
        return st;
    if ((st = make_map_2d(&map_y, Y, (uint64_t)out, (uint64_t)rows, kEpiCols, 32, CU_TENSOR_MAP_SWIZZLE_64B,
                          "Y")) != ELSA_OK)
        return st;

    static std::atomic<bool> attr_set[64][2];   // zero-initialised; a double set by racing threads is harmless
    auto kernel = dtype == ELSA_BF16 ? linear_tc_dense_kernel<true> : linear_tc_dense_kernel<false>;
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
    ProfileScope scope(ELSA_KERNEL_LINEAR_TC_DENSE, stream);
    launch_pdl(kernel, dim3(grid), dim3(kThreads), smem, stream, 1, map_x, map_w, map_y, p);
    return launched("linear_tc_dense");
}

}  // namespace elsa
