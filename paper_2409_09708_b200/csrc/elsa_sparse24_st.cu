// N:M sparse linear (N <= 2) on the 2:4 sparse MMA for long reduction dimensions: the weight streams
// through tensor memory, never through shared memory.
//
// Same product as elsa_sparse24_pair.cu (Sec. 2, Fig. 2 bottom of the ELSA paper, on the 2-of-4
// re-encoding of the packed weight).  At the sparse MMA rate shared memory cannot carry both operands:
// the pair kernel stages the compressed weight tile beside the activations for every row tile and
// runs at about half the sparse rate, and the weight-stationary kernel avoids it only while the whole
// reduction dimension of a 256-feature block fits tensor memory (in <= 896 beside two accumulators).
// Here the block's weight is cut into K chunks of 256.  Loader warps read a chunk from
// global memory (L2-resident image) into registers and write it into one of four tensor-memory
// slots (tcgen05.st: 64 columns of 2-of-4 values, 8 of metadata, per lane = per feature); every
// tcgen05.mma.sp takes its A operand and metadata from the slot, and shared memory carries
// activations only (three stages of 256 of K).  While one slot is multiplied the next ones are being
// written and fetched: a load from L2 takes 1.5-2.5 us under this traffic, several chunk times.
//
// A CTA pair owns a tile of 256 features x 224 token rows (one accumulator of 224 columns beside the
// four slots of 72); tiles of all layers of a launch form one sequence walked with the stride of the
// pairs, feature blocks fastest, so that the pairs that share activation rows read them at the same
// time (once from HBM, then from L2).  With a reduction this long the epilogue's share is small.
//
// Per CTA (576 threads, 96 registers each): warp 0 TMA producer of this CTA's 112 activation rows,
// warp 1 tensor-memory allocation and (leader) MMA issue, warps 2-9 epilogue (two per tensor-memory
// lane quarter, see elsa_sparse24_ws.cu for the transposing stmatrix stores and the lane order of the
// features), warps 10-17 weight loaders (two per lane quarter, taking alternate chunks: the loads of a
// chunk are issued before the wait for its slot, and the next chunk is requested right after the
// tcgen05.st of this one).  The weight image is read in the `tiled` form of nm_to_sp24: rows in the
// permuted lane order, and inside a block of 32 rows x 256 k the 16-byte units of all rows
// interleaved, so that a warp's load is one contiguous run.  Waits are bounded as in the other kernels.

#include <atomic>
#include <mutex>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kFeatPerCta = 128;   // weight rows per CTA = TMEM lanes
constexpr int kPairFeat = 256;     // MMA M over the pair
constexpr int kRowTile = 224;      // token rows per pair tile = MMA N
constexpr int kRowsPerCta = kRowTile / 2;
constexpr int kChunkK = 256;       // logical K per weight slot = per activation stage
constexpr int kSpUmmaK = 32;
constexpr int kSlots = 4;
constexpr int kSlotCols = kChunkK / 4 + kChunkK / 32;   // 64 columns of values + 8 of metadata
constexpr int kSlotCol0 = kRowTile;                     // slots follow the accumulator
constexpr int kTmemCols = 512;
constexpr int kStages = 3;
constexpr int kEpiParts = 2;       // epilogue warps per TMEM lane quarter
constexpr int kEpiWarps = 4 * kEpiParts;
constexpr int kLoaderWarp0 = 2 + kEpiWarps;
constexpr int kLoaderParts = 2;   // loader warps per lane quarter, taking every second chunk each
constexpr int kLoaderWarps = 4 * kLoaderParts;
constexpr int kThreads = (kLoaderWarp0 + kLoaderWarps) * 32;
constexpr int kStepCols = 16;      // token rows per tcgen05.ld / pair of stmatrix
constexpr int kStepsPerWarp = kRowTile / kStepCols / kEpiParts;   // 7
constexpr int kRoundSteps = 4;     // steps an epilogue warp holds in registers at a time
constexpr int kRounds = (kStepsPerWarp + kRoundSteps - 1) / kRoundSteps;
constexpr int kStageBytes = (kChunkK / 64) * kRowsPerCta * 128;   // 64 KB: four quarters of 128 rows x 128 bytes
constexpr int kStagingBytes = 2 * kStepCols * 64;                 // per epilogue warp: two buffers of 16 rows x 32 features
constexpr int kStagingTotal = kEpiWarps * kStagingBytes;
constexpr int kBarrierBytes = 512;

static_assert(kRowTile + kSlots * kSlotCols <= kTmemCols, "accumulator and weight slots fit tensor memory");
static_assert(kStepsPerWarp * kEpiParts * kStepCols == kRowTile, "the epilogue warps cover the tile exactly");
static_assert(kLoaderWarp0 % 4 == 2, "warp & 3 must walk the lane quarters for epilogue and loader warps alike");

// One layer of a launch; lives in kernel-parameter space.
struct alignas(64) StLayer {
    CUtensorMap map_x, map_y;
    const uint8_t* a_img;    // tiled 2-of-4 image (see the head of this file)
    const uint8_t* meta;     // metadata blocks of 2 KB per (128 features, 128 k)
    const uint16_t* bias;
    int rows, out, in;
    int tiles_f;       // ceil(out / 256)
    int tile_begin;    // index of this layer's first tile in the launch's sequence
    int num_chunks;    // ceil(in / 256)
    int num_k_blocks;  // in / 128
    int act;           // epilogue activation (0 none, 1 GELU) on acc + bias
};

constexpr int kGroupMax = 84;   // layers per launch (kernel parameters are limited to 32 KB)

template <int kMaxLayers>
struct StGroup {
    StLayer layer[kMaxLayers];
    int n_layers;
    int num_tiles;
    uint32_t idesc;
    uint32_t* dev_status;
};

// (22 warps are allocated as 24: 80 registers per thread is what the register file allows, and a loader warp
// holds a whole chunk, 72 of them, between its loads and its tensor-memory stores)
// kAct: the instantiation whose epilogue applies the layer's activation (single-layer launches).
template <bool kBf16, int kMaxLayers, bool kAct>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_sp24_st_kernel(const __grid_constant__ StGroup<kMaxLayers> p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;

    const uint32_t staging_base = smem_base + (uint32_t)(kStages * kStageBytes);
    const uint32_t bar_off = (uint32_t)(kStages * kStageBytes) + kStagingTotal;
    const uint32_t bar_base = smem_base + bar_off;
    const uint32_t full_bar = bar_base;                          // leader only
    const uint32_t empty_bar = bar_base + 8 * kStages;           // per CTA
    const uint32_t a_full_bar = bar_base + 16 * kStages;         // leader only: a weight slot is written in both CTAs
    const uint32_t a_empty_bar = a_full_bar + 8 * kSlots;        // per CTA: the MMAs that read a slot are done
    const uint32_t tmem_full_bar = a_empty_bar + 8 * kSlots;     // per CTA
    const uint32_t tmem_empty_bar = tmem_full_bar + 8;           // leader only
    const uint32_t holder_off = bar_off + 16 * kStages + 16 * kSlots + 16;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(a_full_bar + 8 * s, 2 * 4);   // one loader warp per lane quarter and CTA
            mbar_init(a_empty_bar + 8 * s, 1);
        }
        mbar_init(tmem_full_bar, 1);
        mbar_init(tmem_empty_bar, 2 * kEpiWarps);
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
        // ------------------------------------------------ producer: this CTA's half of the activation rows
        // (whole warp converged, one elected lane issues).  One 3-D copy per stage brings the four 64-wide K
        // quarters of the chunk: [quarter][row][128 bytes]; quarters beyond `in` arrive as zeros.
        const bool elected = elect_one();
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        int cur = 0;
        for (int tile = pair; ok && tile < p.num_tiles; tile += num_pairs) {
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            const StLayer& L = p.layer[cur];
            const int t = tile - L.tile_begin;
            const int r0 = (t / L.tiles_f) * kRowTile + (int)cta_rank * kRowsPerCta;
            for (int c = 0; c < L.num_chunks; ++c) {
                ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                const uint32_t dst = smem_base + (uint32_t)(stage * kStageBytes);
                const uint32_t bar = mapa_shared(full_bar + 8 * stage, 0);
                if (elected) {
                    if (cta_rank == 0) mbar_arrive_expect_tx(full_bar + 8 * stage, (uint32_t)(2 * kStageBytes));
                    tma_load_3d_pair(dst, &L.map_x, bar, 0, r0, (kChunkK / 64) * c);
                }
                __syncwarp();
                if (++stage == kStages) { stage = 0; phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop and waits on the barriers; one elected lane issues, through the
        // predicate inside each instruction's asm block.
        if (cta_rank == 0) {
            const uint32_t elected = elect_one() ? 1u : 0u;
            const uint32_t tmem_u = __reduce_or_sync(0xFFFFFFFFu, tmem_base);
            const uint32_t idesc = p.idesc;
            constexpr uint32_t quarter = (uint32_t)(kRowsPerCta * 128) >> 4;   // descriptor units between K quarters
            int stage = 0, slot = 0;
            uint32_t phase = 0, a_phase = 0, acc_phase = 0;
            bool ok = true;
            int cur = 0;
            for (int tile = pair; ok && tile < p.num_tiles; tile += num_pairs) {
                while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
                const int num_chunks = p.layer[cur].num_chunks;
                const bool half_tail = (p.layer[cur].in % kChunkK) != 0;     // the last chunk holds 128 of K only
                ok = mbar_wait(tmem_empty_bar, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                for (int c = 0; c < num_chunks; ++c) {
                    ok = mbar_wait(a_full_bar + 8 * slot, a_phase, abort_flag, p.dev_status, 7);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t b_desc0 = smem_desc_k_major_sw128(smem_base + (uint32_t)(stage * kStageBytes));
                    const uint32_t a_col = tmem_u + (uint32_t)(kSlotCol0 + slot * kSlotCols);
                    const uint32_t e_col = a_col + (uint32_t)(kChunkK / 4);
                    if (half_tail && c == num_chunks - 1) {
#pragma unroll
                        for (int j = 0; j < kChunkK / kSpUmmaK / 2; ++j) {
                            const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)(j >> 1) * quarter + 4u * (uint32_t)(j & 1));
                            umma_sp_f16_pair_ts(tmem_u, a_col + (uint32_t)(8 * j), b_desc, e_col + (uint32_t)j, idesc,
                                                (uint32_t)((c | j) != 0), elected);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < kChunkK / kSpUmmaK; ++j) {
                            const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)(j >> 1) * quarter + 4u * (uint32_t)(j & 1));
                            umma_sp_f16_pair_ts(tmem_u, a_col + (uint32_t)(8 * j), b_desc, e_col + (uint32_t)j, idesc,
                                                (uint32_t)((c | j) != 0), elected);
                        }
                    }
                    umma_commit_pair_if(empty_bar + 8 * stage, 3, elected);     // stage and slot are free once these MMAs are done
                    umma_commit_pair_if(a_empty_bar + 8 * slot, 3, elected);
                    if (++stage == kStages) { stage = 0; phase ^= 1u; }
                    if (++slot == kSlots) { slot = 0; a_phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair_if(tmem_full_bar, 3, elected);
                acc_phase ^= 1u;
            }
        }
        __syncwarp();
    } else if (warp >= kLoaderWarp0) {
        // ------------------------------------------------ weight loaders: lanes are features
        // Image row (block base + TMEM lane) is the row of the feature the lane holds.
        // A global load takes about as long as the MMAs of two chunks, so one warp per quarter cannot keep up:
        // two take every second chunk of the pair's chunk sequence each.
        const int q = warp & 3;
        const int part = (warp - kLoaderWarp0) >> 2;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t a_full_remote = mapa_shared(a_full_bar, 0);
        // position in the pair's chunk sequence
        int tile = pair, c = 0, cur = 0, slot = 0, turn = 0;
        uint32_t a_phase = 0;
        bool have = tile < p.num_tiles;
        if (have)
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
        auto step = [&]() {
            if (++slot == kSlots) { slot = 0; a_phase ^= 1u; }
            if (++turn == kLoaderParts) turn = 0;
            if (++c == p.layer[cur].num_chunks) {
                c = 0;
                tile += num_pairs;
                if (tile >= p.num_tiles) { have = false; return; }
                while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            }
        };
        while (have && turn != part) step();

        uint32_t v[4][16];
        uint32_t e[2][4];
        // 16 + 2 loads of 16 bytes per lane for the chunk at (tile, c), all in flight together
        auto request = [&]() {
            const StLayer& L = p.layer[cur];
            const int t = tile - L.tile_begin;
            const int ft128 = (t % L.tiles_f) * 2 + (int)cta_rank;
            const int row32 = ft128 * 4 + q;                          // block of 32 image rows this warp feeds
            const bool rows_ok = row32 * 32 < L.out;                  // a started block of 32 exists (zeros past out)
            const bool blk_ok = ft128 * kFeatPerCta < L.out;
            const int kc = L.in - c * kChunkK < kChunkK ? L.in - c * kChunkK : kChunkK;   // 256, or 128 in a tail
            // 8 KB per (block of 32 rows, chunk) = 512 units of 16 bytes
            const uint4* src = reinterpret_cast<const uint4*>(L.a_img + (size_t)row32 * 32 * (size_t)L.in) + (size_t)c * (kChunkK * 2) + lane;
            const uint4* e_blk = reinterpret_cast<const uint4*>(L.meta) +
                                 ((size_t)(blk_ok ? ft128 : 0) * (size_t)L.num_k_blocks + (size_t)(2 * c)) * 128 + (size_t)(q * 32 + lane);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    uint4 u = make_uint4(0u, 0u, 0u, 0u);
                    if (rows_ok && (4 * j + i) * 16 < kc) u = __ldg(src + (4 * j + i) * 32);
                    v[j][4 * i] = u.x; v[j][4 * i + 1] = u.y; v[j][4 * i + 2] = u.z; v[j][4 * i + 3] = u.w;
                }
            }
#pragma unroll
            for (int b = 0; b < 2; ++b) {
                uint4 u = make_uint4(0u, 0u, 0u, 0u);
                if (blk_ok && b * 128 < kc) u = __ldg(e_blk + (size_t)b * 128);
                e[b][0] = u.x; e[b][1] = u.y; e[b][2] = u.z; e[b][3] = u.w;
            }
        };
        if (have) request();
        bool ok = true;
        while (have && ok) {
            // The chunk was requested before its slot is waited for, and the next one is requested as soon as
            // this one has gone to tensor memory: a load is always in flight under the MMAs.
            const int my_slot = slot;
            ok = mbar_wait(a_empty_bar + 8 * my_slot, a_phase ^ 1u, abort_flag, p.dev_status, 8);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t a_col = lane_base + (uint32_t)(kSlotCol0 + my_slot * kSlotCols);
#pragma unroll
            for (int j = 0; j < 4; ++j) tmem_st_32x32b_x16(a_col + (uint32_t)(16 * j), v[j]);
#pragma unroll
            for (int b = 0; b < 2; ++b) tmem_st_32x32b_x4(a_col + (uint32_t)(kChunkK / 4 + 4 * b), e[b]);
            do { step(); } while (have && turn != part);
            if (have) request();
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            // tcgen05.wait::st has completed the writes and tensor memory is not ordinary memory: the arrival
            // needs no cluster-scope release (which would also wait for everything else this warp has in flight)
            if (lane == 0) mbar_arrive_cluster(a_full_remote + 8 * my_slot);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue: lanes are features, columns are token rows
        const int q = warp & 3;                 // TMEM lane quarter this warp may touch
        const int part = (warp - 2) >> 2;       // which of the quarter's warps
        const uint32_t empty_remote = mapa_shared(tmem_empty_bar, 0);
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        uint32_t acc_phase = 0;
        const uint32_t buf0 = staging_base + (uint32_t)((warp - 2) * kStagingBytes);
        // lane t holds feature 8 * (t % 4) + t / 4 of the quarter's 32 (see elsa_sparse24_ws.cu)
        const int feat_in_quarter = 8 * (lane & 3) + (lane >> 2);
        const uint32_t st_off = (uint32_t)((2 * (lane >> 3) + (lane & 1)) * 64 + ((lane & 7) >> 1) * 16);
        // this warp's run of token columns: kStepsPerWarp steps of 16 from first_step
        const int first_step = part * kStepsPerWarp;
        uint32_t store_count = 0;

        int cur = 0;
        for (int tile = pair; tile < p.num_tiles; tile += num_pairs) {
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            const StLayer& L = p.layer[cur];
            const int t = tile - L.tile_begin;
            const int f0 = ((t % L.tiles_f) * 2 + (int)cta_rank) * kFeatPerCta + q * 32;
            const int row0 = (t / L.tiles_f) * kRowTile + first_step * kStepCols;
            const int f = f0 + feat_in_quarter;
            const int l_rows = L.rows, l_out = L.out;
            const float bias_f = (L.bias != nullptr && f < l_out) ? bias_to_float<kBf16>(__ldg(L.bias + f)) : 0.f;
            const int l_act = kAct ? L.act : 0;
            (void)l_act;
            bool ok = mbar_wait(tmem_full_bar, acc_phase, abort_flag, p.dev_status, 4);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_col = lane_base + (uint32_t)(first_step * kStepCols);
            // Rounds of three steps (registers): the next round is requested before the current one is stored,
            // and the accumulator goes back to the MMA warp as soon as the last round has arrived.
            // Staging: rows of 32 features (64 bytes, no swizzle), two buffers of one step per warp.
            uint32_t rr[kRoundSteps][16];
            auto store_step = [&](int s, const uint32_t (&w)[8]) {
                const uint32_t buf = buf0 + (store_count & 1u) * (uint32_t)(kStepCols * 64);
                if (lane == 0) bulk_wait_group_read<1>();   // the store two steps ago has drained this buffer
                __syncwarp();
                stmatrix_x4_trans(buf + st_off, w[0], w[1], w[2], w[3]);
                stmatrix_x4_trans(buf + st_off + 512, w[4], w[5], w[6], w[7]);
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (f0 < l_out && row0 + s * kStepCols < l_rows) tma_store_2d(&L.map_y, buf, f0, row0 + s * kStepCols);
                    bulk_commit_group();
                }
                ++store_count;
            };
#pragma unroll
            for (int i = 0; i < kRoundSteps; ++i)
                if (i < kStepsPerWarp) tmem_ld_32x32b_x16(t_col + (uint32_t)(i * kStepCols), rr[i]);
            tmem_wait_ld();
#pragma unroll
            for (int rd = 0; rd < kRounds; ++rd) {
                uint32_t w[kRoundSteps][8];
#pragma unroll
                for (int i = 0; i < kRoundSteps; ++i)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        w[i][j] = kAct ? pack2<kBf16>(apply_act(__uint_as_float(rr[i][2 * j]) + bias_f, l_act),
                                                      apply_act(__uint_as_float(rr[i][2 * j + 1]) + bias_f, l_act))
                                       : pack2<kBf16>(__uint_as_float(rr[i][2 * j]) + bias_f, __uint_as_float(rr[i][2 * j + 1]) + bias_f);
                if (rd + 1 < kRounds) {
#pragma unroll
                    for (int i = 0; i < kRoundSteps; ++i)
                        if ((rd + 1) * kRoundSteps + i < kStepsPerWarp)
                            tmem_ld_32x32b_x16(t_col + (uint32_t)(((rd + 1) * kRoundSteps + i) * kStepCols), rr[i]);
                }
                // the last round's values are waited for, and the accumulator handed back, before this round is
                // stored: the MMA warp should not wait for stores
                if (rd + 2 == kRounds) tmem_wait_ld();
                if (rd + 2 == kRounds || kRounds == 1) {       // every column of the accumulator has been read
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(empty_remote);
                }
#pragma unroll
                for (int i = 0; i < kRoundSteps; ++i)
                    if (rd * kRoundSteps + i < kStepsPerWarp) store_step(rd * kRoundSteps + i, w[i]);
                if (rd + 1 < kRounds && rd + 2 != kRounds) tmem_wait_ld();
            }
            acc_phase ^= 1u;
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

template <bool kBf16, int kMaxLayers, bool kAct>
elsa_status launch_st_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status, cudaStream_t stream,
                            const DeviceInfo& dev)
{
    auto kernel = linear_tc_sp24_st_kernel<kBf16, kMaxLayers, kAct>;
    const size_t smem = (size_t)kStages * kStageBytes + kStagingTotal + kBarrierBytes + 1024;
    if (smem > dev.smem_optin) return fail(ELSA_ERR_CUDA, "not enough shared memory for the streaming sparse kernel");

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
        cfg.dynamicSmemBytes = dev.smem_optin;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int m = 0;
        if (cudaOccupancyMaxActiveClusters(&m, kernel, &cfg) != cudaSuccess || m < 1) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaOccupancyMaxActiveClusters: %s", cudaGetErrorString(e));
        }
        max_pairs[slot].store(m, std::memory_order_release);
    }

    static StGroup<kMaxLayers> g;   // host staging of the kernel parameters
    static std::mutex g_mutex;
    std::lock_guard<std::mutex> lock(g_mutex);
    int tile_begin = 0;
    for (int i = 0; i < n; ++i) {
        const SparseJob& j = jobs[i];
        StLayer& L = g.layer[i];
        if (j.in % 128 != 0) return fail(ELSA_ERR_SHAPE, "in=%d does not fit the streaming sparse kernel", j.in);
        L.rows = j.rows; L.out = j.out; L.in = j.in;
        L.tiles_f = (j.out + kPairFeat - 1) / kPairFeat;
        L.tile_begin = tile_begin;
        tile_begin += L.tiles_f * ((j.rows + kRowTile - 1) / kRowTile);
        L.num_chunks = (j.in + kChunkK - 1) / kChunkK;
        L.num_k_blocks = j.in / 128;
        L.bias = j.bias;
        L.act = j.act;
        L.a_img = (const uint8_t*)j.workspace;
        L.meta = (const uint8_t*)j.workspace + sp24_meta_offset(j.out, j.in);
        elsa_status st;
        if ((st = make_map_x_quarters(&L.map_x, j.X, (uint64_t)j.in, (uint64_t)j.rows, kRowsPerCta, kChunkK / 64)) != ELSA_OK) return st;
        if ((st = make_map_2d(&L.map_y, j.Y, (uint64_t)j.out, (uint64_t)j.rows, 32, kStepCols, CU_TENSOR_MAP_SWIZZLE_NONE,
                              "Y")) != ELSA_OK)
            return st;
    }
    g.n_layers = n;
    g.num_tiles = tile_begin;
    g.dev_status = dev_status;
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    // sparse flag, fp32 accumulate, A and B of type fmt, K-major, N = 256, M = 256 over the pair
    g.idesc = (1u << 2) | (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(kRowTile >> 3) << 17) |
              ((uint32_t)(kPairFeat >> 4) << 24);

    const int pairs = g.num_tiles < max_pairs[slot].load(std::memory_order_acquire) ? g.num_tiles : max_pairs[slot].load(std::memory_order_acquire);
    ProfileScope scope(ELSA_KERNEL_LINEAR_TC_SP24_ST, stream);
    cudaError_t e = launch_pdl(kernel, dim3((unsigned)(2 * pairs)), dim3(kThreads), smem, stream, 2, g);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ELSA_ERR_CUDA, "launch of linear_tc_sp24_st failed: %s", cudaGetErrorString(e));
    }
    return launched("linear_tc_sp24_st");
}

}  // namespace

int linear_tc_sparse_st_group_max() { return kGroupMax; }

bool linear_tc_sparse_st_suits(int in, int N) { return linear_tc_sparse_suits(in, N) && in % 128 == 0; }

elsa_status launch_linear_tc_sparse_st_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                             cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (n < 1 || n > kGroupMax) return fail(ELSA_ERR_SHAPE, "a grouped launch carries 1 to %d layers, got %d", kGroupMax, n);
    bool act = false;
    for (int i = 0; i < n; ++i) act = act || jobs[i].act != 0;
    if (act) {
        // layers with an activation in the epilogue run one per launch, on the instantiation that has it
        for (int i = 0; i < n; ++i) {
            st = dtype == ELSA_BF16 ? launch_st_group<true, 1, true>(jobs + i, 1, dtype, dev_status, stream, dev)
                                    : launch_st_group<false, 1, true>(jobs + i, 1, dtype, dev_status, stream, dev);
            if (st != ELSA_OK) return st;
        }
        return ELSA_OK;
    }
    if (n == 1)
        return dtype == ELSA_BF16 ? launch_st_group<true, 1, false>(jobs, 1, dtype, dev_status, stream, dev)
                                  : launch_st_group<false, 1, false>(jobs, 1, dtype, dev_status, stream, dev);
    return dtype == ELSA_BF16 ? launch_st_group<true, kGroupMax, false>(jobs, n, dtype, dev_status, stream, dev)
                              : launch_st_group<false, kGroupMax, false>(jobs, n, dtype, dev_status, stream, dev);
}

elsa_status launch_linear_tc_sparse_st(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                       const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype, uint16_t* Y,
                                       void* workspace, uint32_t* dev_status, cudaStream_t stream)
{
    if (!linear_tc_sparse_st_suits(in, N) || N == M)
        return fail(ELSA_ERR_NM, "level %d:%d with in=%d does not fit the streaming sparse kernel", N, M, in);
    uint16_t* a_img = (uint16_t*)workspace;
    uint8_t* meta = (uint8_t*)workspace + sp24_meta_offset(out, in);
    elsa_status st = launch_nm_to_sp24(vals, idx, out, in, N, M, 128, SP24_TILED, a_img, meta, stream);
    if (st != ELSA_OK) return st;
    SparseJob job;
    job.X = X; job.bias = bias; job.Y = Y; job.workspace = workspace;
    job.rows = rows; job.in = in; job.out = out;
    return launch_linear_tc_sparse_st_group(&job, 1, dtype, dev_status, stream);
}

}  // namespace elsa
