// N:M sparse linear (N <= 2) on the 2:4 sparse MMA with the weight held in tensor memory.
//
// Same product as elsa_sparse24_pair.cu (Sec. 2, Fig. 2 bottom of the ELSA paper, on the 2-of-4
// re-encoding of the packed weight).  That kernel streams the compressed weight tile and its metadata
// through shared memory again for every tile of token rows, and at the sparse MMA rate the weight and
// activation bytes together exceed what shared memory can deliver per cycle.  Here the weight does
// not move: a CTA pair owns one block of 256 output features of a layer for the whole layer.  Its
// 2-of-4 values (in/4 columns) and metadata (in/32 columns) are written once into the tensor memory
// of the two CTAs and every tcgen05.mma.sp reads its A operand from there; shared memory carries
// activations only.  What is left of tensor memory holds TWO accumulators of `nt` token rows each
// (144 for in = 768), so the epilogue of one tile runs under the MMAs of the next.  Narrow MMAs only
// pay because the issuing lane is predicated inside the instruction's own asm block: a branch around
// each tcgen05.mma costs the issuing warp about 80 cycles per instruction, the predicated form under
// 40, and a sparse MMA over 144 token rows lasts 72.
//
// Schedule of a layer over P pairs: F = ceil(out / 256) feature blocks, G = P / F row groups.  Pair p
// takes feature block p % F and the row tiles g, g + G, g + 2G, ... with g = p / F, so the F pairs
// of a group read the same activation rows at about the same time (one fetch from HBM, the rest from
// L2).  Pairs beyond G * F sit the layer out.  A launch may carry several layers; each pair walks
// them in order, reloading its weight block at every layer.
//
// Per CTA: warp 0 TMA producer for this CTA's half of the activation rows; warp 1 tensor-memory
// allocation and, in the leader, MMA issue; twelve epilogue warps (three per tensor-memory lane
// quarter, each with its own run of token columns) write the weight block into tensor memory at the
// start of a layer and run the epilogue.  The accumulator is transposed (lanes are features, columns
// are token rows) and Y is row-major, so the epilogue has to turn a lane's column pair into a row's
// feature run.  stmatrix with .trans does that in one instruction per 8 x 32 outputs if lane t of a
// quarter holds feature 8 * (t % 4) + t / 4 of its 32; the weight image is therefore built with its
// rows in that order (SP24_PERMUTED form of nm_to_sp24), and only the bias index and the store address
// here know about it.  Waits are bounded as in the other kernels.

#include <atomic>
#include <mutex>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kFeatPerCta = 128;   // weight rows per CTA = TMEM lanes
constexpr int kPairFeat = 256;     // MMA M over the pair
constexpr int kBlockK = 128;       // granularity of `in` (one metadata block)
constexpr int kStageK = 256;       // logical K per pipeline stage: eight MMAs per barrier round trip
constexpr int kSpUmmaK = 32;
constexpr int kNumAccum = 2;
constexpr int kTmemCols = 512;
constexpr int kMaxIn = 1024;       // in / 4 + in / 32 + 2 * nt columns must fit 512
constexpr int kMaxStages = 8;
constexpr int kEpiParts = 3;       // epilogue warps per TMEM lane quarter
constexpr int kEpiWarps = 4 * kEpiParts;
constexpr int kThreads = 64 + kEpiWarps * 32;
constexpr int kStepCols = 16;      // token rows per tcgen05.ld / pair of stmatrix
constexpr int kMaxSteps = 4;       // steps per epilogue warp and tile
constexpr int kMaxRowTile = kStepCols * kMaxSteps * kEpiParts;   // 192 token rows per pair tile (MMA N)
constexpr int kStagingBytes = kMaxSteps * kStepCols * 64;        // per epilogue warp: rows of 32 features
constexpr int kStagingTotal = kEpiWarps * kStagingBytes;
constexpr int kBarrierBytes = 512;

struct alignas(64) WsLayer {
    CUtensorMap map_x, map_y;
    const uint16_t* a_img;   // 2-of-4 values [out rounded up to 32][in / 2], rows in the permuted order
    const uint8_t* meta;     // metadata blocks of 2 KB per (128 features, 128 k)
    const uint16_t* bias;
    int rows, out, in;
    int nt;            // token rows per pair tile
    int steps_per_warp;   // 16-column steps each epilogue warp of a quarter takes
    int tiles_f;       // F
    int groups;        // G
    int row_tiles;     // ceil(rows / nt)
    uint32_t idesc;
    int act;           // epilogue activation (0 none, 1 GELU) on acc + bias
};

constexpr int kGroupMax = 92;   // layers per launch (kernel parameters are limited to 32 KB)

template <int kMaxLayers>
struct WsGroup {
    WsLayer layer[kMaxLayers];
    int n_layers;
    int stages;
    int stage_bytes;   // one pipeline stage: kStageK / 64 quarters of (largest nt / 2) rows of 128 bytes
    uint32_t* dev_status;
};

// kAct: the instantiation whose epilogue applies the layer's activation (single-layer launches).
template <bool kBf16, int kMaxLayers, bool kAct>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_sp24_ws_kernel(const __grid_constant__ WsGroup<kMaxLayers> p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1;

    const uint32_t staging_base = smem_base + (uint32_t)(p.stages * p.stage_bytes);
    const uint32_t bar_off = (uint32_t)(p.stages * p.stage_bytes) + kStagingTotal;
    const uint32_t bar_base = smem_base + bar_off;
    const uint32_t full_bar = bar_base;                       // leader only
    const uint32_t empty_bar = bar_base + 8 * kMaxStages;     // per CTA
    const uint32_t tmem_full_bar = bar_base + 16 * kMaxStages;        // per CTA
    const uint32_t tmem_empty_bar = tmem_full_bar + 8 * kNumAccum;    // leader only
    const uint32_t w_ready_bar = tmem_empty_bar + 8 * kNumAccum;      // leader only
    const uint32_t layer_bar = w_ready_bar + 8;                       // per CTA: epilogue warps between layers
    const uint32_t holder_off = bar_off + 16 * kMaxStages + 16 * kNumAccum + 16;
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
        mbar_init(w_ready_bar, 2 * kEpiWarps);
        mbar_init(layer_bar, kEpiWarps);
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
        // (whole warp converged, one elected lane issues: see the MMA warp).  One 3-D copy per stage
        // brings the four 64-wide K quarters of the stage: [quarter][row][128 bytes]; quarters beyond `in`
        // (a last stage of 128) arrive as zeros and are not multiplied.
        {
            const bool elected = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int li = 0; ok && li < p.n_layers; ++li) {
                const WsLayer& L = p.layer[li];
                if (pair >= L.groups * L.tiles_f) continue;
                const int half_rows = L.nt >> 1;
                const uint32_t tx_bytes = (uint32_t)(2 * (kStageK / 64) * half_rows * 128);   // both CTAs' boxes, in full
                const int num_k_stages = (L.in + kStageK - 1) / kStageK;
                for (int r = pair / L.tiles_f; ok && r < L.row_tiles; r += L.groups) {
                    const int r0 = r * L.nt + (int)cta_rank * half_rows;
                    for (int ks = 0; ks < num_k_stages; ++ks) {
                        ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                        ok = __all_sync(0xFFFFFFFFu, ok);
                        if (!ok) break;
                        const uint32_t dst = smem_base + (uint32_t)(stage * p.stage_bytes);
                        const uint32_t bar = mapa_shared(full_bar + 8 * stage, 0);
                        if (elected) {
                            if (cta_rank == 0) mbar_arrive_expect_tx(full_bar + 8 * stage, tx_bytes);
                            tma_load_3d_pair(dst, &L.map_x, bar, 0, r0, (kStageK / 64) * ks);
                        }
                        __syncwarp();
                        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop and waits on the barriers; one elected lane issues, through a
        // predicate inside each instruction's asm block.  With the warp converged the descriptors stay in
        // uniform registers and no branch surrounds the instruction: measured ~36 cycles per MMA, against
        // ~80 with `if (elected)` around it and more with a single thread inside a divergent branch.
        if (cta_rank == 0) {
            const uint32_t elected = elect_one() ? 1u : 0u;
            // the base address was read from shared memory into an ordinary register; a warp reduction
            // returns it in a uniform one, so that every address derived from it stays uniform too
            const uint32_t tmem_u = __reduce_or_sync(0xFFFFFFFFu, tmem_base);
            int stage = 0;
            uint32_t phase = 0;
            int acc = 0;
            uint32_t acc_phase = 0;
            uint32_t w_phase = 0;
            bool ok = true;
            for (int li = 0; ok && li < p.n_layers; ++li) {
                const WsLayer& L = p.layer[li];
                if (pair >= L.groups * L.tiles_f) continue;
                const int g = pair / L.tiles_f;
                if (g >= L.row_tiles) continue;
                // the weight block of this layer is in tensor memory (both CTAs)
                ok = mbar_wait(w_ready_bar, w_phase, abort_flag, p.dev_status, 7);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                w_phase ^= 1u;
                tc_fence_after();
                const uint32_t a_col0 = tmem_u + (uint32_t)(kNumAccum * L.nt);
                const uint32_t e_col0 = a_col0 + (uint32_t)(L.in >> 2);
                const uint32_t idesc = L.idesc;
                const int num_k_stages = (L.in + kStageK - 1) / kStageK;
                const bool half_tail = (L.in % kStageK) != 0;      // the last stage holds 128 of K only
                const uint32_t quarter = (uint32_t)(L.nt * 64) >> 4;   // descriptor units between K quarters
                for (int r = g; ok && r < L.row_tiles; r += L.groups) {
                    ok = mbar_wait(tmem_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_u + (uint32_t)(acc * L.nt);
                    for (int ks = 0; ks < num_k_stages; ++ks) {
                        ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                        ok = __all_sync(0xFFFFFFFFu, ok);
                        if (!ok) break;
                        tc_fence_after();
                        const uint64_t b_desc0 = smem_desc_k_major_sw128(smem_base + (uint32_t)(stage * p.stage_bytes));
                        const uint32_t a_col = a_col0 + (uint32_t)(ks * 8 * (kStageK / kSpUmmaK));
                        const uint32_t e_col = e_col0 + (uint32_t)(ks * (kStageK / kSpUmmaK));
                        // operands are computed by the whole warp (they stay uniform); only the instruction
                        // itself is predicated on the elected lane
                        if (half_tail && ks == num_k_stages - 1) {
#pragma unroll
                            for (int j = 0; j < kStageK / kSpUmmaK / 2; ++j) {
                                const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)(j >> 1) * quarter + 4u * (uint32_t)(j & 1));
                                umma_sp_f16_pair_ts(d_tmem, a_col + (uint32_t)(8 * j), b_desc, e_col + (uint32_t)j, idesc,
                                                    (uint32_t)((ks | j) != 0), elected);
                            }
                        } else {
#pragma unroll
                            for (int j = 0; j < kStageK / kSpUmmaK; ++j) {
                                const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)(j >> 1) * quarter + 4u * (uint32_t)(j & 1));
                                umma_sp_f16_pair_ts(d_tmem, a_col + (uint32_t)(8 * j), b_desc, e_col + (uint32_t)j, idesc,
                                                    (uint32_t)((ks | j) != 0), elected);
                            }
                        }
                        umma_commit_pair_if(empty_bar + 8 * stage, 3, elected);
                        if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                    }
                    if (!ok) break;
                    umma_commit_pair_if(tmem_full_bar + 8 * acc, 3, elected);
                    if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ weight loader + epilogue: lanes are features
        const int q = warp & 3;                 // TMEM lane quarter this warp may touch
        const int part = (warp - 2) >> 2;       // which of the quarter's warps
        const uint32_t empty_remote = mapa_shared(tmem_empty_bar, 0);
        const uint32_t w_ready_remote = mapa_shared(w_ready_bar, 0);
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t layer_phase = 0;
        const uint32_t buf = staging_base + (uint32_t)((warp - 2) * kStagingBytes);
        // Lane t holds feature 8 * (t % 4) + t / 4 of the quarter's 32.  The staging buffer is rows of 32
        // features (64 bytes, no swizzle); one stmatrix.x4.trans writes 8 token rows: lane t gives the
        // address of (row 2 * (t / 8) + (t & 1), features 8 * ((t % 8) / 2) ...), and the two rows of a
        // matrix are 128 consecutive bytes, so no two of its addresses share a bank.
        const int feat_in_quarter = 8 * (lane & 3) + (lane >> 2);
        const uint32_t st_addr = buf + (uint32_t)((2 * (lane >> 3) + (lane & 1)) * 64 + ((lane & 7) >> 1) * 16);

        bool ok = true;
        bool first_layer = true;
        for (int li = 0; ok && li < p.n_layers; ++li) {
            const WsLayer& L = p.layer[li];
            if (pair >= L.groups * L.tiles_f) continue;
            const int g = pair / L.tiles_f;
            if (g >= L.row_tiles) continue;
            const int ft128 = (pair % L.tiles_f) * 2 + (int)cta_rank;
            const int f0 = ft128 * kFeatPerCta + q * 32;
            const int f = f0 + feat_in_quarter;
            const int l_rows = L.rows, l_out = L.out, nt = L.nt;
            const bool f_ok = f < l_out;

            // The column ranges of accumulators and weight block depend on the layer, and the warps of a
            // quarter read different columns of the same lanes: nobody writes the new weight block before
            // every epilogue warp of this CTA has read its last accumulator of the previous layer.
            if (!first_layer) {
                __syncwarp();
                if (lane == 0) mbar_arrive(layer_bar);
                ok = mbar_wait(layer_bar, layer_phase, abort_flag, p.dev_status, 8);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                layer_phase ^= 1u;
            }
            first_layer = false;

            // ---- this warp's share of the weight block into tensor memory.  Every MMA of the previous
            // layer has completed: this warp waited for the accumulator of that layer's last tile.  Image
            // row (block base + TMEM lane) is already the row of the feature this lane holds.
            {
                const uint32_t a_col0 = lane_base + (uint32_t)(kNumAccum * nt);
                const uint32_t e_col0 = a_col0 + (uint32_t)(L.in >> 2);
                const uint4* a_row = reinterpret_cast<const uint4*>(L.a_img + (size_t)(ft128 * kFeatPerCta + q * 32 + lane) * (size_t)(L.in >> 1));
                const bool blk_ok = ft128 * kFeatPerCta < l_out;     // rows of a started block of 32 exist (zero beyond out)
                const bool row_ok = f0 < l_out;
                const int a_chunks = L.in >> 6;          // 16 columns (64 bytes) each
                for (int c = part; c < a_chunks; c += kEpiParts) {
                    uint32_t v[16];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        uint4 t = make_uint4(0u, 0u, 0u, 0u);
                        if (row_ok) t = __ldg(a_row + 4 * c + i);
                        v[4 * i] = t.x; v[4 * i + 1] = t.y; v[4 * i + 2] = t.z; v[4 * i + 3] = t.w;
                    }
                    tmem_st_32x32b_x16(a_col0 + (uint32_t)(16 * c), v);
                }
                const uint4* e_blk = reinterpret_cast<const uint4*>(L.meta) +
                                     (size_t)(blk_ok ? ft128 : 0) * (size_t)(L.in / kBlockK) * 128 + (size_t)(q * 32 + lane);
                for (int kb = part; kb < L.in / kBlockK; kb += kEpiParts) {
                    uint4 t = make_uint4(0u, 0u, 0u, 0u);
                    if (blk_ok) t = __ldg(e_blk + (size_t)kb * 128);
                    uint32_t v[4] = {t.x, t.y, t.z, t.w};
                    tmem_st_32x32b_x4(e_col0 + (uint32_t)(4 * kb), v);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster_release(w_ready_remote);
            }
            const float bias_f = (L.bias != nullptr && f_ok) ? bias_to_float<kBf16>(__ldg(L.bias + f)) : 0.f;
            const int l_act = kAct ? L.act : 0;
            (void)l_act;
            // this warp's run of token columns: steps of 16, [first_step, first_step + my_steps)
            const int total_steps = nt / kStepCols;
            const int first_step = part * L.steps_per_warp;
            int my_steps = total_steps - first_step;
            if (my_steps > L.steps_per_warp) my_steps = L.steps_per_warp;
            if (my_steps < 0) my_steps = 0;

            for (int r = g; r < L.row_tiles; r += L.groups) {
                const int row0 = r * nt + first_step * kStepCols;
                ok = mbar_wait(tmem_full_bar + 8 * acc, acc_phase, abort_flag, p.dev_status, 4);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_col = lane_base + (uint32_t)(acc * nt + first_step * kStepCols);
                // all of this warp's columns are requested at once and the accumulator goes back to the MMA
                // warp before anything is converted
                uint32_t rr[kMaxSteps][16];
#pragma unroll
                for (int s = 0; s < kMaxSteps; ++s)
                    if (s < my_steps) tmem_ld_32x32b_x16(t_col + (uint32_t)(s * kStepCols), rr[s]);
                if (my_steps > 0) tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive_cluster(empty_remote + 8 * acc);
                    bulk_wait_group_read<0>();   // the stores of the previous tile have drained the buffer
                }
                __syncwarp();
#pragma unroll
                for (int s = 0; s < kMaxSteps; ++s) {
                    if (s >= my_steps) continue;
                    uint32_t w[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        w[j] = kAct ? pack2<kBf16>(apply_act(__uint_as_float(rr[s][2 * j]) + bias_f, l_act),
                                                   apply_act(__uint_as_float(rr[s][2 * j + 1]) + bias_f, l_act))
                                    : pack2<kBf16>(__uint_as_float(rr[s][2 * j]) + bias_f, __uint_as_float(rr[s][2 * j + 1]) + bias_f);
                    stmatrix_x4_trans(st_addr + (uint32_t)(s * kStepCols * 64), w[0], w[1], w[2], w[3]);
                    stmatrix_x4_trans(st_addr + (uint32_t)(s * kStepCols * 64 + 512), w[4], w[5], w[6], w[7]);
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (f0 < l_out) {
#pragma unroll
                        for (int s = 0; s < kMaxSteps; ++s)
                            if (s < my_steps && row0 + s * kStepCols < l_rows)
                                tma_store_2d(&L.map_y, buf + (uint32_t)(s * kStepCols * 64), f0, row0 + s * kStepCols);
                    }
                    bulk_commit_group();
                }
                if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
            }
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

// Token rows per pair tile for a layer of this input width: the largest multiple of 16, at most
// kMaxRowTile, such that two accumulators fit beside the weight block and its metadata; 0 if none does.
int ws_row_tile(int in)
{
    const int left = kTmemCols - in / 4 - in / 32;
    int nt = left / kNumAccum / kStepCols * kStepCols;
    if (nt > kMaxRowTile) nt = kMaxRowTile;
    return nt >= 64 ? nt : 0;
}

template <bool kBf16, int kMaxLayers, bool kAct>
elsa_status launch_ws_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status, cudaStream_t stream,
                            const DeviceInfo& dev)
{
    auto kernel = linear_tc_sp24_ws_kernel<kBf16, kMaxLayers, kAct>;
    const int fixed = kStagingTotal + kBarrierBytes + 1024;
    int max_nt = 0;
    for (int i = 0; i < n; ++i) {
        const int nt = ws_row_tile(jobs[i].in);
        if (nt > max_nt) max_nt = nt;
    }
    if (max_nt == 0) return fail(ELSA_ERR_SHAPE, "in=%d does not fit the weight-stationary sparse kernel", jobs[0].in);
    // a stage slot is sized for the widest row tile of the launch, so that narrow tiles still keep
    // the same number of activation bytes in flight
    const int stage_bytes = (kStageK / 64) * (max_nt / 2) * 128;
    int stages = (int)((dev.smem_optin - fixed) / stage_bytes);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(ELSA_ERR_CUDA, "not enough shared memory for two pipeline stages");
    const size_t smem = (size_t)stages * stage_bytes + fixed;

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
    const int pairs = max_pairs[slot].load(std::memory_order_acquire);

    static WsGroup<kMaxLayers> g;   // host staging of the kernel parameters
    static std::mutex g_mutex;
    std::lock_guard<std::mutex> lock(g_mutex);
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    int used_pairs = 0;
    for (int i = 0; i < n; ++i) {
        const SparseJob& j = jobs[i];
        WsLayer& L = g.layer[i];
        L.nt = ws_row_tile(j.in);
        L.tiles_f = (j.out + kPairFeat - 1) / kPairFeat;
        if (L.nt == 0 || j.in % kBlockK != 0 || L.tiles_f > pairs)
            return fail(ELSA_ERR_SHAPE, "in=%d out=%d does not fit the weight-stationary sparse kernel", j.in, j.out);
        L.rows = j.rows; L.out = j.out; L.in = j.in;
        L.steps_per_warp = (L.nt / kStepCols + kEpiParts - 1) / kEpiParts;
        L.row_tiles = (j.rows + L.nt - 1) / L.nt;
        L.groups = pairs / L.tiles_f;
        if (L.groups > L.row_tiles) L.groups = L.row_tiles;
        if (L.groups * L.tiles_f > used_pairs) used_pairs = L.groups * L.tiles_f;
        L.bias = j.bias;
        L.act = j.act;
        L.a_img = (const uint16_t*)j.workspace;
        L.meta = (const uint8_t*)j.workspace + sp24_meta_offset(j.out, j.in);
        // sparse flag, fp32 accumulate, A and B of type fmt, K-major, N = nt, M = 256 over the pair
        L.idesc = (1u << 2) | (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(L.nt >> 3) << 17) |
                  ((uint32_t)(kPairFeat >> 4) << 24);
        elsa_status st;
        if ((st = make_map_x_quarters(&L.map_x, j.X, (uint64_t)j.in, (uint64_t)j.rows, (uint32_t)(L.nt / 2), kStageK / 64)) != ELSA_OK) return st;
        if ((st = make_map_2d(&L.map_y, j.Y, (uint64_t)j.out, (uint64_t)j.rows, 32, kStepCols, CU_TENSOR_MAP_SWIZZLE_NONE,
                              "Y")) != ELSA_OK)
            return st;
    }
    g.n_layers = n;
    g.stages = stages;
    g.stage_bytes = stage_bytes;
    g.dev_status = dev_status;

    ProfileScope scope(ELSA_KERNEL_LINEAR_TC_SP24_WS, stream);
    cudaError_t e = launch_pdl(kernel, dim3((unsigned)(2 * used_pairs)), dim3(kThreads), smem, stream, 2, g);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ELSA_ERR_CUDA, "launch of linear_tc_sp24_ws failed: %s", cudaGetErrorString(e));
    }
    return launched("linear_tc_sp24_ws");
}

}  // namespace

int linear_tc_sparse_ws_group_max() { return kGroupMax; }

bool linear_tc_sparse_ws_suits(int in, int out, int N, int sm_count)
{
    return linear_tc_sparse_suits(in, N) && in % kBlockK == 0 && in <= kMaxIn && ws_row_tile(in) != 0 &&
           (out + kPairFeat - 1) / kPairFeat <= sm_count / 2;
}

elsa_status launch_linear_tc_sparse_ws_group(const SparseJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
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
            st = dtype == ELSA_BF16 ? launch_ws_group<true, 1, true>(jobs + i, 1, dtype, dev_status, stream, dev)
                                    : launch_ws_group<false, 1, true>(jobs + i, 1, dtype, dev_status, stream, dev);
            if (st != ELSA_OK) return st;
        }
        return ELSA_OK;
    }
    if (n == 1)
        return dtype == ELSA_BF16 ? launch_ws_group<true, 1, false>(jobs, 1, dtype, dev_status, stream, dev)
                                  : launch_ws_group<false, 1, false>(jobs, 1, dtype, dev_status, stream, dev);
    return dtype == ELSA_BF16 ? launch_ws_group<true, kGroupMax, false>(jobs, n, dtype, dev_status, stream, dev)
                              : launch_ws_group<false, kGroupMax, false>(jobs, n, dtype, dev_status, stream, dev);
}

elsa_status launch_linear_tc_sparse_ws(const uint16_t* X, int rows, const uint16_t* vals, const uint32_t* idx,
                                       const uint16_t* bias, int out, int in, int N, int M, elsa_dtype dtype, uint16_t* Y,
                                       void* workspace, uint32_t* dev_status, cudaStream_t stream)
{
    elsa_status st = launch_linear_tc_sparse_pair_prepare(vals, idx, out, in, N, M, SP24_PERMUTED, workspace, stream);
    if (st != ELSA_OK) return st;
    SparseJob job;
    job.X = X; job.bias = bias; job.Y = Y; job.workspace = workspace;
    job.rows = rows; job.in = in; job.out = out;
    return launch_linear_tc_sparse_ws_group(&job, 1, dtype, dev_status, stream);
}

}  // namespace elsa
