// Tensor-core linear for sm_100a on CTA pairs: Y[rows][out] = X[rows][in] * Wd[out][in]^T + bias.
//
// Same contraction as elsa_linear_tc.cu (the product step of Sec. 2, Fig. 2 bottom of the ELSA paper,
// on the weight image the MMA reads), restructured around the limit that kernel ran into: a
// single-CTA 128 x 256 x 16 MMA reads 12 KB of operands from shared memory in 128 cycles and TMA
// writes as much, 192 B/clk against the SM's 128 B/clk.  Here two CTAs on neighbouring SMs form a
// cluster and share one tile of 256 rows x BN features: each CTA stages its own 128 rows of X and
// only half of the W rows, and one tcgen05.mma.cta_group::2 (M = 256) issued by the leader CTA
// drives both tensor cores, so each SM moves 2/3 of the bytes per MMA.
//
// Per CTA (352 threads):
//   warp 0      TMA producer for this CTA's operand halves; completion bytes of both CTAs are
//               credited to the leader's stage barrier
//   warp 1      allocates tensor memory (pair-wide); in the leader one lane issues the MMAs and
//               commits, by multicast, onto both CTAs' stage and accumulator barriers
//   warps 2-9   epilogue, two warps per TMEM lane quarter (alternating 32-column chunks):
//               tcgen05.ld of all the warp's chunks, accumulator released, then + bias in fp32,
//               round to 16 bit, swizzled staging, TMA store
//   warp 10     bias loader: copies the next tile's bias into one of two shared buffers, so the
//               epilogue warps issue no global loads of their own
// Two TMEM accumulators let the MMAs of tile i+1 overlap the epilogue of tile i.  Every wait is
// bounded; on expiry ELSA_ERR_TIMEOUT is recorded and all roles of the CTA leave; a cluster barrier
// before tensor memory is released keeps either CTA from leaving while its partner may still read
// its shared memory.

#include <atomic>
#include <mutex>

#include "elsa_tc_common.cuh"

#include <type_traits>

namespace elsa {
namespace {

constexpr int kRowsPerCta = 128;   // rows of X per CTA = TMEM lanes
constexpr int kPairRows = 256;     // MMA M over the pair
constexpr int kBlockK = 64;
constexpr int kUmmaK = 16;
constexpr int kMaxBlockN = 256;
constexpr int kNumAccum = 2;
constexpr int kTmemCols = kNumAccum * kMaxBlockN;
constexpr int kMaxStages = 8;
constexpr int kEpiWarps = 8;
constexpr int kEpiParts = kEpiWarps / 4;   // warps per TMEM lane quarter; they share the quarter's chunks
constexpr int kBiasWarp = 2 + kEpiWarps;
constexpr int kThreads = (kBiasWarp + 1) * 32;
constexpr int kEpiCols = 32;
constexpr int kMaxChunksPerWarp = kMaxBlockN / kEpiCols / kEpiParts;
constexpr int kATileBytes = kRowsPerCta * kBlockK * 2;
constexpr int kStagingBytes = 32 * kEpiCols * 2;
constexpr int kStagingBufs = 1;     // one staging buffer per epilogue warp: the shared memory goes to a sixth pipeline stage instead
constexpr int kStagingTotal = kEpiWarps * kStagingBufs * kStagingBytes;
constexpr int kBiasBytes = 2 * kMaxBlockN * 2;   // two tiles' bias as stored (16 bit)
constexpr int kScaleBytes = 2 * kMaxBlockN * 4;  // INT8 form: two tiles' combined scales (fp32)
constexpr int kBarrierBytes = 256;

// One layer of a launch.  A launch may carry several layers (a group): the persistent CTA pairs walk the
// tiles of all of them in one sequence, so the tail of one layer overlaps the head of the next and
// only one kernel ramp is paid.  All of it lives in kernel-parameter space.
struct alignas(64) PairLayer {
    CUtensorMap map_x, map_w, map_y;
    int rows, out;
    int bn;            // features per pair tile (MMA N)
    int tiles_n;
    int tile_begin;    // index of this layer's first tile in the launch's sequence
    int num_k_blocks;
    uint32_t idesc;
    const uint16_t* bias;
    const float* w_scale;   // INT8 form only: per-feature weight scale, and the activations' scale
    float x_scale;
    int act;                    // epilogue activation (0 none, 1 GELU) on acc + bias
    const uint16_t* residual;   // [rows][out] added after the activation, or NULL
};

template <int kMaxLayers>
struct PairGroup {
    PairLayer layer[kMaxLayers];
    int n_layers;
    int num_tiles;     // over all layers
    int stages;
    uint32_t* dev_status;
    // Tn form only (one layer per launch): the reduction is cut into `splits` ranges of K blocks, a tile index t is
    // tile t / splits over range t % splits, and each range's fp32 sums go to partial[range][rows][out].
    int splits;
    float* partial;
};

constexpr int kStageBytesMax = kATileBytes + (kMaxBlockN / 2) * kBlockK * 2;   // stage slots sized for BN = 256
// Forms of the kernel: plain (acc + bias), INT8 (integer operands, scaled in the epilogue), fused (activation and
// residual added in the epilogue), Tn (both operands stored with the reduction index outermost: A [K][M] and
// B [K][N], the weight-gradient product dY^T X; tiles arrive as boxes of 64 features x 64 reduction rows and the
// MMA reads them through MN-major descriptors). Separate instantiations, so the plain form pays nothing for the
// others.
constexpr int kFormPlain = 0, kFormInt8 = 1, kFormFused = 2, kFormTn = 3;
constexpr int kTnBoxBytes = 64 * 64 * 2;   // one box of the Tn form: 64 reduction rows of 128 bytes
constexpr int kGroupMax = 72;   // layers per grouped launch (kernel parameters are limited to 32 KB)

// kInt8: operands are signed 8-bit integers (rows of 128 elements per 128-byte swizzle row, K = 32 per MMA,
// int32 accumulators); the epilogue turns an accumulator into float, multiplies by x_scale * w_scale[feature],
// adds the bias, each in fp32 with one rounding per operation, and rounds once to the 16-bit output type.
template <bool kBf16, int kForm, int kMaxLayers>
__global__ void __launch_bounds__(kThreads, 1)
linear_tc_pair_kernel(const __grid_constant__ PairGroup<kMaxLayers> p)
{
    constexpr bool kInt8 = kForm == kFormInt8;     // 8-bit integer operands, scales in the epilogue
    constexpr bool kFused = kForm == kFormFused;   // activation and residual in the epilogue
    constexpr bool kTn = kForm == kFormTn;         // operands [K][M] and [K][N]

    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const uint32_t cta_rank = cluster_ctarank();       // 0 = leader of the pair
    const int pair = blockIdx.x >> 1;
    const int num_pairs = gridDim.x >> 1;
    constexpr int stage_bytes = kStageBytesMax;

    const uint32_t staging_base = smem_base + (uint32_t)(p.stages * stage_bytes);
    const uint32_t bias_off = (uint32_t)(p.stages * stage_bytes) + kStagingTotal;
    const uint32_t scale_off = bias_off + kBiasBytes;
    const uint32_t bar_base = smem_base + scale_off + kScaleBytes;
    const uint32_t full_bar = bar_base;                       // used in the leader only
    const uint32_t empty_bar = bar_base + 8 * kMaxStages;     // per CTA
    const uint32_t tmem_full_bar = bar_base + 16 * kMaxStages;                 // per CTA
    const uint32_t tmem_empty_bar = tmem_full_bar + 8 * kNumAccum;             // used in the leader only
    const uint32_t bias_full_bar = tmem_empty_bar + 8 * kNumAccum;             // per CTA
    const uint32_t bias_empty_bar = bias_full_bar + 16;                        // per CTA
    const uint32_t holder_off = scale_off + kScaleBytes + 16 * kMaxStages + 16 * kNumAccum + 32;
    volatile uint32_t* tmem_holder = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_gen + holder_off + 4);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full_bar + 8 * s, 1);
            mbar_init(empty_bar + 8 * s, 1);
        }
        for (int a = 0; a < kNumAccum; ++a) {
            mbar_init(tmem_full_bar + 8 * a, 1);
            mbar_init(tmem_empty_bar + 8 * a, 2 * kEpiWarps);   // every epilogue warp of both CTAs
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bias_full_bar + 8 * b, 1);
            mbar_init(bias_empty_bar + 8 * b, kEpiWarps);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async_smem();
    }
    if (warp == 1) tmem_alloc_pair(smem_base + holder_off, kTmemCols);
    tc_fence_before();
    __syncthreads();
    // both CTAs' barriers exist and both allocations are done before either CTA signals the other
    cluster_arrive();
    cluster_wait();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    // set-up above touched no global memory; from here on the predecessor's writes are needed
    pdl_wait_for_predecessors();
    pdl_release_successors();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer (both CTAs)
        // The whole warp walks the loop and waits; one elected lane issues (see the MMA warp).
        {
            const bool elected = elect_one();
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            int cur = 0;
            for (int tile = pair; ok && tile < p.num_tiles; tile += num_pairs) {
                while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
                const PairLayer& L = p.layer[cur];
                int t = tile - L.tile_begin;
                int kb0 = 0, kb1 = L.num_k_blocks;
                if constexpr (kTn) {
                    const int range = t % p.splits;
                    t /= p.splits;
                    kb0 = (int)((long long)L.num_k_blocks * range / p.splits);
                    kb1 = (int)((long long)L.num_k_blocks * (range + 1) / p.splits);
                }
                const int half_bn = L.bn >> 1;
                const int m0 = (t / L.tiles_n) * kPairRows + (int)cta_rank * kRowsPerCta;
                const int n0 = (t % L.tiles_n) * L.bn + (int)cta_rank * half_bn;
                const uint32_t tx_bytes = (uint32_t)(2 * (kATileBytes + half_bn * kBlockK * 2));
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(empty_bar + 8 * stage, phase ^ 1u, abort_flag, p.dev_status, 1);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    const uint32_t a_dst = smem_base + (uint32_t)(stage * stage_bytes);
                    const uint32_t bar = mapa_shared(full_bar + 8 * stage, 0);
                    if (elected) {
                        // the leader's stage barrier collects the bytes of both CTAs
                        if (cta_rank == 0) mbar_arrive_expect_tx(full_bar + 8 * stage, tx_bytes);
                        // a stage is 128 bytes of K per row: 64 16-bit or 128 8-bit elements
                        if constexpr (kTn) {
                            // boxes of 64 features x 64 reduction rows, 8 KB each: this CTA's 128 rows of A and its
                            // half of B's columns
                            for (int i = 0; i < kRowsPerCta / 64; ++i)
                                tma_load_2d_pair(a_dst + (uint32_t)(i * kTnBoxBytes), &L.map_x, bar, m0 + 64 * i, kb * kBlockK);
                            for (int i = 0; i < half_bn / 64; ++i)
                                tma_load_2d_pair(a_dst + kATileBytes + (uint32_t)(i * kTnBoxBytes), &L.map_w, bar, n0 + 64 * i, kb * kBlockK);
                        } else {
                            tma_load_2d_pair(a_dst, &L.map_x, bar, kb * (kInt8 ? 2 * kBlockK : kBlockK), m0);
                            tma_load_2d_pair(a_dst + kATileBytes, &L.map_w, bar, kb * (kInt8 ? 2 * kBlockK : kBlockK), n0);
                        }
                    }
                    __syncwarp();
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer (leader CTA only)
        // The whole warp walks the loop and waits on the barriers with its operands in uniform
        // registers; only the MMA and commit instructions are predicated on one elected lane.  A
        // single thread inside a divergent branch needs about twice as long to issue one MMA.
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
                int kb0 = 0, kb1 = p.layer[cur].num_k_blocks;
                if constexpr (kTn) {
                    const int range = (tile - p.layer[cur].tile_begin) % p.splits;
                    kb0 = (int)((long long)p.layer[cur].num_k_blocks * range / p.splits);
                    kb1 = (int)((long long)p.layer[cur].num_k_blocks * (range + 1) / p.splits);
                }
                const uint32_t idesc = p.layer[cur].idesc;
                ok = mbar_wait(tmem_empty_bar + 8 * acc, acc_phase ^ 1u, abort_flag, p.dev_status, 2);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_u + (uint32_t)(acc * kMaxBlockN);
                for (int kb = kb0; kb < kb1; ++kb) {
                    ok = mbar_wait(full_bar + 8 * stage, phase, abort_flag, p.dev_status, 3);
                    ok = __all_sync(0xFFFFFFFFu, ok);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = smem_base + (uint32_t)(stage * stage_bytes);
                    const uint64_t a_desc = kTn ? smem_desc_mn_major_sw128(a_addr, kTnBoxBytes) : smem_desc_k_major_sw128(a_addr);
                    const uint64_t b_desc = kTn ? smem_desc_mn_major_sw128(a_addr + kATileBytes, kTnBoxBytes)
                                                : smem_desc_k_major_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        if constexpr (kTn)
                            // 16 reduction rows of 128 bytes per MMA: the start address moves by 2048 bytes
                            umma_f16_pair_if(d_tmem, a_desc + (uint64_t)(k * (kUmmaK * 128 >> 4)), b_desc + (uint64_t)(k * (kUmmaK * 128 >> 4)),
                                             idesc, (uint32_t)(kb != kb0 || k != 0), elected);
                        else if constexpr (kInt8)
                            umma_i8_pair_if(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                            (uint32_t)((kb | k) != 0), elected);
                        else
                            umma_f16_pair_if(d_tmem, a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), idesc,
                                             (uint32_t)((kb | k) != 0), elected);
                    }
                    umma_commit_pair_if(empty_bar + 8 * stage, 3, elected);   // frees this stage in both CTAs
                    if (++stage == p.stages) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                umma_commit_pair_if(tmem_full_bar + 8 * acc, 3, elected);     // accumulator complete in both CTAs
                if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
            }
        }
        __syncwarp();
    } else if (warp == kBiasWarp) {
        // ------------------------------------------------ bias loader: tile i + 1's bias while tile i is stored
        // (kept out of the epilogue warps: a global load in flight there holds up their proxy fences)
        int cur = 0;
        uint32_t it = 0;
        for (int tile = pair; tile < p.num_tiles; tile += num_pairs, ++it) {
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            const PairLayer& L = p.layer[cur];
            const int n0 = (((tile - L.tile_begin) / (kTn ? p.splits : 1)) % L.tiles_n) * L.bn;
            const uint32_t b = it & 1u;
            bool ok = mbar_wait(bias_empty_bar + 8 * b, ((it >> 1) & 1u) ^ 1u, abort_flag, p.dev_status, 5);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            const uint16_t* l_bias = L.bias;
            for (int j = lane; j < L.bn; j += 32) {
                const int o = n0 + j;
                const uint16_t v = (l_bias != nullptr && o < L.out) ? __ldg(l_bias + o) : (uint16_t)0;
                asm volatile("st.shared.b16 [%0], %1;" ::"r"(smem_base + bias_off + b * (kMaxBlockN * 2) + (uint32_t)(j * 2)), "h"(v)
                             : "memory");
                if constexpr (kInt8) {
                    const float sc = o < L.out ? __fmul_rn(L.x_scale, __ldg(L.w_scale + o)) : 0.f;
                    asm volatile("st.shared.b32 [%0], %1;" ::"r"(smem_base + scale_off + b * (kMaxBlockN * 4) + (uint32_t)(j * 4)),
                                 "r"(__float_as_uint(sc))
                                 : "memory");
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bias_full_bar + 8 * b);
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ epilogue (warps 2..9)
        const int q = warp & 3;                 // TMEM lane quarter this warp may read
        const int ew = warp - 2;                // private staging slot
        const int part = ew >> 2;               // which of the quarter's warps: chunks part, part + kEpiParts, ...
        const uint32_t stage_buf = staging_base + (uint32_t)(ew * kStagingBufs * kStagingBytes);
        const uint32_t empty_remote = mapa_shared(tmem_empty_bar, 0);
        int acc = 0;
        uint32_t acc_phase = 0;
        uint32_t chunk_counter = 0;
        int cur = 0;
        uint32_t it = 0;

        for (int tile = pair; tile < p.num_tiles; tile += num_pairs, ++it) {
            while (cur + 1 < p.n_layers && tile >= p.layer[cur + 1].tile_begin) ++cur;
            const PairLayer& L = p.layer[cur];
            int t = tile - L.tile_begin;
            int range = 0;
            if constexpr (kTn) {
                range = t % p.splits;
                t /= p.splits;
            }
            (void)range;
            const int chunks = L.bn / kEpiCols;
            const int my_chunks = (chunks - part + kEpiParts - 1) / kEpiParts;
            const int m0 = (t / L.tiles_n) * kPairRows + (int)cta_rank * kRowsPerCta;
            const int n0 = (t % L.tiles_n) * L.bn;
            const int l_rows = L.rows, l_out = L.out;
            const uint32_t bias_b = it & 1u;
            const uint32_t bias_cur = smem_base + bias_off + bias_b * (kMaxBlockN * 2);
            const uint32_t scale_cur = smem_base + scale_off + bias_b * (kMaxBlockN * 4);
            (void)scale_cur;
            const int l_act = kFused ? L.act : 0;
            const uint16_t* l_res = kFused ? L.residual : nullptr;
            (void)l_act;
            (void)l_res;
            bool ok = mbar_wait(bias_full_bar + 8 * bias_b, (it >> 1) & 1u, abort_flag, p.dev_status, 6);
            ok = ok && mbar_wait(tmem_full_bar + 8 * acc, acc_phase, abort_flag, p.dev_status, 4);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * kMaxBlockN);
            const int row0 = m0 + q * 32;

            // converts, stages and stores one 32 x 32 chunk
            auto emit = [&](const uint32_t (&r)[32], int c) {
                if constexpr (kTn) {
                    if (p.partial != nullptr) {
                        // a range's fp32 sums as they are: this lane's row, 32 consecutive columns
                        const int row = row0 + lane, col0 = n0 + c * kEpiCols;
                        if (row < l_rows) {
                            float4* dst = reinterpret_cast<float4*>(p.partial + ((size_t)range * (size_t)l_rows + row) * (size_t)l_out + col0);
#pragma unroll
                            for (int v = 0; v < 8; ++v)
                                if (col0 + 4 * v < l_out)
                                    dst[v] = make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                                         __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                        }
                        return;
                    }
                }
                // 16 columns: + bias (read as stored, eight values per load), rounded to 16 bit
                auto convert16 = [&](auto with_act, int h, uint32_t (&pk)[8]) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        uint32_t bw[4];
                        asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(bw[0]), "=r"(bw[1]), "=r"(bw[2]), "=r"(bw[3])
                                     : "r"(bias_cur + (uint32_t)(c * kEpiCols * 2 + (2 * h + g) * 16)));
                        // this lane's row of the residual, eight values (a whole load lies inside or outside the row)
                        uint32_t res[4] = {0u, 0u, 0u, 0u};
                        if constexpr (kFused) {
                            if (l_res != nullptr) {
                                const int row = row0 + lane;
                                const int col = n0 + c * kEpiCols + (2 * h + g) * 8;
                                if (row < l_rows && col < l_out) {
                                    const uint4 u = __ldg(reinterpret_cast<const uint4*>(l_res + (size_t)row * (size_t)l_out + col));
                                    res[0] = u.x; res[1] = u.y; res[2] = u.z; res[3] = u.w;
                                }
                            }
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 bv = raw2_to_float2<kBf16>(bw[e]);
                            const int j = 8 * h + 4 * g + e;
                            if constexpr (kInt8) {
                                float sx, sy;
                                asm volatile("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(sx), "=f"(sy)
                                             : "r"(scale_cur + (uint32_t)((c * kEpiCols + 2 * j) * 4)));
                                const float vx = __fadd_rn(__fmul_rn((float)(int)r[2 * j], sx), bv.x);
                                const float vy = __fadd_rn(__fmul_rn((float)(int)r[2 * j + 1], sy), bv.y);
                                pk[4 * g + e] = pack2<kBf16>(vx, vy);
                            } else {
                                float vx = __uint_as_float(r[2 * j]) + bv.x;
                                float vy = __uint_as_float(r[2 * j + 1]) + bv.y;
                                if constexpr (kFused) {
                                    const float2 rv = raw2_to_float2<kBf16>(res[e]);   // zeros without a residual
                                    if constexpr (decltype(with_act)::value) {
                                        vx = gelu_exact(vx);
                                        vy = gelu_exact(vy);
                                    }
                                    vx += rv.x;
                                    vy += rv.y;
                                }
                                pk[4 * g + e] = pack2<kBf16>(vx, vy);
                            }
                        }
                    }
                };
                const uint32_t buf = stage_buf + (chunk_counter % kStagingBufs) * kStagingBytes;
                const uint32_t row_addr = buf + (uint32_t)(lane * 64);
                const uint32_t sw = (uint32_t)((lane >> 1) & 3);   // 64-byte swizzle of the staging rows
                uint32_t pk[8];
                // the activation is a warp-uniform property of the layer: one branch per chunk, none per value
                if (kFused && l_act == 1) convert16(std::true_type{}, 0, pk);
                else convert16(std::false_type{}, 0, pk);
                if (lane == 0) bulk_wait_group_read<kStagingBufs - 1>();   // the store that last used this buffer has drained it
                __syncwarp();
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h == 1) {
                        if (kFused && l_act == 1) convert16(std::true_type{}, 1, pk);
                        else convert16(std::false_type{}, 1, pk);
                    }
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(row_addr + (((uint32_t)(2 * h + j) ^ sw) << 4)),
                                     "r"(pk[4 * j]), "r"(pk[4 * j + 1]), "r"(pk[4 * j + 2]), "r"(pk[4 * j + 3])
                                     : "memory");
                    }
                }
                fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    const int col0 = n0 + c * kEpiCols;
                    if (row0 < l_rows && col0 < l_out) tma_store_2d(&L.map_y, buf, col0, row0);
                    bulk_commit_group();
                }
                ++chunk_counter;
            };
            // hands the accumulator back once this warp's last load of it has completed
            auto release = [&]() {
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(empty_remote + 8 * acc);
            };

            // All of this warp's chunks are requested at once and the accumulator is handed back as soon
            // as they have arrived: a tensor-memory load queues behind the MMAs already issued, so
            // loads taken one at a time would each pay that wait.
            uint32_t r[kMaxChunksPerWarp][32];
#pragma unroll
            for (int i = 0; i < kMaxChunksPerWarp; ++i)
                if (i < my_chunks) tmem_ld_32x32b_x32(t_row + (uint32_t)((part + kEpiParts * i) * kEpiCols), r[i]);
            tmem_wait_ld();
            release();
#pragma unroll
            for (int i = 0; i < kMaxChunksPerWarp; ++i)
                if (i < my_chunks) emit(r[i], part + kEpiParts * i);
            // this warp has read the tile's bias for the last time
            __syncwarp();
            if (lane == 0) mbar_arrive(bias_empty_bar + 8 * bias_b);
            if (++acc == kNumAccum) { acc = 0; acc_phase ^= 1u; }
        }
        if (lane == 0) bulk_wait_group_all();
        __syncwarp();
    }

    // ------------------------------------------------ teardown
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // a wait gave up: let copies and MMAs that may still be in flight land first
        for (int i = 0; i < 200; ++i) __nanosleep(10000);
    }
    // neither CTA leaves, or frees tensor memory, while its partner may still use its shared memory
    cluster_arrive();
    cluster_wait();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

// Width of a pair tile in output features.  Cost model: the tiles run in waves over the SM pairs, a tile costs
// its width plus a fixed share (operand staging, pipeline fill), and features past `out` in the last tile are
// wasted work; among equals the widest wins (fewest re-reads of X).  For the large layers this picks 256 or
// the width that divides `out`; below a wave of tiles it narrows the tile until the pairs are occupied.
int pick_pair_block_n(int out, int rows, int sm_count, bool whole_boxes = false)
{
    const int pairs = sm_count / 2 > 0 ? sm_count / 2 : 1;
    const long long row_tiles = (rows + kPairRows - 1) / kPairRows;
    int best = 64;
    long long best_cost = -1;
    const int cand[4] = {256, 192, 128, 64};
    for (int i = 0; i < 4; ++i) {
        const int bn = cand[i];
        if (whole_boxes && bn % 128 != 0) continue;   // the Tn form loads each CTA's half in boxes of 64 features
        const long long tiles = row_tiles * ((out + bn - 1) / bn);
        const long long waves = (tiles + pairs - 1) / pairs;
        const long long cost = waves * (bn + 32);
        if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
    }
    return best;
}

}  // namespace

bool linear_tc_pair_suits(int rows, int out, int sm_count)
{
    // worth pairing CTAs only when there are enough 256-row tiles to occupy every SM pair
    const int bn = pick_pair_block_n(out, rows, sm_count);
    const long long tiles = (long long)((rows + kPairRows - 1) / kPairRows) * ((out + bn - 1) / bn);
    return tiles >= sm_count / 2;
}

namespace {

template <bool kBf16, int kForm, int kMaxLayers>
elsa_status launch_group(const PairJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status, cudaStream_t stream,
                         const DeviceInfo& dev)
{
    constexpr bool kInt8 = kForm == kFormInt8;
    static PairGroup<kMaxLayers> g;   // host staging of the kernel parameters (single-threaded launch path)
    static std::mutex g_mutex;
    std::lock_guard<std::mutex> lock(g_mutex);
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    int tile_begin = 0;
    for (int i = 0; i < n; ++i) {
        const PairJob& j = jobs[i];
        PairLayer& L = g.layer[i];
        L.rows = j.rows; L.out = j.out;
        L.bn = (kForm == kFormTn && j.splits > 1) ? 256 : pick_pair_block_n(j.out, j.rows, dev.sm_count, kForm == kFormTn);
        L.tiles_n = (j.out + L.bn - 1) / L.bn;
        L.tile_begin = tile_begin;
        tile_begin += ((j.rows + kPairRows - 1) / kPairRows) * L.tiles_n * (kForm == kFormTn ? j.splits : 1);
        L.bias = j.bias;
        L.w_scale = j.w_scale;
        L.x_scale = j.x_scale;
        L.act = j.act;
        L.residual = j.residual;
        elsa_status st;
        if constexpr (kInt8) {
            L.num_k_blocks = (j.in + 2 * kBlockK - 1) / (2 * kBlockK);
            // int32 accumulate, A and B signed 8-bit, K-major, N = bn, M = 256 over the pair
            L.idesc = (2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(L.bn >> 3) << 17) | ((uint32_t)(kPairRows >> 4) << 24);
            if ((st = make_map_2d_u8(&L.map_x, j.X, (uint64_t)j.in, (uint64_t)j.rows, 2 * kBlockK, kRowsPerCta,
                                     CU_TENSOR_MAP_SWIZZLE_128B, "X")) != ELSA_OK)
                return st;
            if ((st = make_map_2d_u8(&L.map_w, j.Wd, (uint64_t)j.in, (uint64_t)j.out, 2 * kBlockK, (uint32_t)(L.bn / 2),
                                     CU_TENSOR_MAP_SWIZZLE_128B, "W")) != ELSA_OK)
                return st;
        } else if constexpr (kForm == kFormTn) {
            // A = j.X [in][rows] and B = j.Wd [in][out], `in` the reduction: both MN-major (bits 15 and 16)
            L.num_k_blocks = (j.in + kBlockK - 1) / kBlockK;
            L.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(L.bn >> 3) << 17) |
                      ((uint32_t)(kPairRows >> 4) << 24);
            if ((st = make_map_2d(&L.map_x, j.X, (uint64_t)j.rows, (uint64_t)j.in, 64, kBlockK, CU_TENSOR_MAP_SWIZZLE_128B,
                                  "A")) != ELSA_OK)
                return st;
            if ((st = make_map_2d(&L.map_w, j.Wd, (uint64_t)j.out, (uint64_t)j.in, 64, kBlockK, CU_TENSOR_MAP_SWIZZLE_128B,
                                  "B")) != ELSA_OK)
                return st;
        } else {
            L.num_k_blocks = (j.in + kBlockK - 1) / kBlockK;
            L.idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(L.bn >> 3) << 17) | ((uint32_t)(kPairRows >> 4) << 24);
            if ((st = make_map_2d(&L.map_x, j.X, (uint64_t)j.in, (uint64_t)j.rows, kBlockK, kRowsPerCta,
                                  CU_TENSOR_MAP_SWIZZLE_128B, "X")) != ELSA_OK)
                return st;
            if ((st = make_map_2d(&L.map_w, j.Wd, (uint64_t)j.in, (uint64_t)j.out, kBlockK, (uint32_t)(L.bn / 2),
                                  CU_TENSOR_MAP_SWIZZLE_128B, "W")) != ELSA_OK)
                return st;
        }
        if ((st = make_map_2d(&L.map_y, j.Y, (uint64_t)j.out, (uint64_t)j.rows, kEpiCols, 32, CU_TENSOR_MAP_SWIZZLE_64B,
                              "Y")) != ELSA_OK)
            return st;
    }
    g.n_layers = n;
    g.splits = kForm == kFormTn ? jobs[0].splits : 1;
    g.partial = kForm == kFormTn && jobs[0].splits > 1 ? jobs[0].partial : nullptr;
    g.num_tiles = tile_begin;
    g.dev_status = dev_status;

    const int fixed = kStagingTotal + kBiasBytes + kScaleBytes + kBarrierBytes + 1024;
    int stages = (int)((dev.smem_optin - fixed) / kStageBytesMax);
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return fail(ELSA_ERR_CUDA, "not enough shared memory for two pipeline stages");
    g.stages = stages;
    const size_t smem = (size_t)stages * kStageBytesMax + fixed;

    auto kernel = linear_tc_pair_kernel<kBf16, kForm, kMaxLayers>;
    static std::atomic<int> max_pairs[64];   // zero-initialised; racing first calls compute the same value
    const int slot = dev.device & 63;
    if (max_pairs[slot].load(std::memory_order_acquire) == 0) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dev.smem_optin) !=
            cudaSuccess) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        // how many CTA pairs the device can hold at once: the persistent schedule assumes all run together
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
    ProfileScope scope(kInt8 ? ELSA_KERNEL_LINEAR_TC_PAIR_I8 : ELSA_KERNEL_LINEAR_TC_PAIR, stream);
    cudaError_t e = launch_pdl(kernel, dim3((unsigned)(2 * pairs)), dim3(kThreads), smem, stream, 2, g);
    if (e != cudaSuccess) {
        cudaGetLastError();
        return fail(ELSA_ERR_CUDA, "launch of linear_tc_pair failed: %s", cudaGetErrorString(e));
    }
    return launched("linear_tc_pair");
}

}  // namespace

int linear_tc_pair_group_max() { return kGroupMax; }

elsa_status launch_linear_tc_pair_group(const PairJob* jobs, int n, elsa_dtype dtype, uint32_t* dev_status,
                                        cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (n < 1 || n > kGroupMax) return fail(ELSA_ERR_SHAPE, "a grouped launch carries 1 to %d layers, got %d", kGroupMax, n);
    bool fused = false;
    for (int i = 0; i < n; ++i) fused = fused || jobs[i].act != 0 || jobs[i].residual != nullptr;
    if (fused) {
        if (n == 1)
            return dtype == ELSA_BF16 ? launch_group<true, kFormFused, 1>(jobs, 1, dtype, dev_status, stream, dev)
                                      : launch_group<false, kFormFused, 1>(jobs, 1, dtype, dev_status, stream, dev);
        return dtype == ELSA_BF16 ? launch_group<true, kFormFused, kGroupMax>(jobs, n, dtype, dev_status, stream, dev)
                                  : launch_group<false, kFormFused, kGroupMax>(jobs, n, dtype, dev_status, stream, dev);
    }
    if (n == 1)
        return dtype == ELSA_BF16 ? launch_group<true, kFormPlain, 1>(jobs, 1, dtype, dev_status, stream, dev)
                                  : launch_group<false, kFormPlain, 1>(jobs, 1, dtype, dev_status, stream, dev);
    return dtype == ELSA_BF16 ? launch_group<true, kFormPlain, kGroupMax>(jobs, n, dtype, dev_status, stream, dev)
                              : launch_group<false, kFormPlain, kGroupMax>(jobs, n, dtype, dev_status, stream, dev);
}

// How many ranges the reduction of an m x n product is cut into: with 256 x 256 tiles, as many as keep one wave of
// work units on the SM pairs (1 when the tiles alone fill them).
int linear_tc_pair_tn_splits(int m, int n, int k, int sm_count)
{
    const int pairs = sm_count / 2 > 0 ? sm_count / 2 : 1;
    const long long tiles = (long long)((m + kPairRows - 1) / kPairRows) * ((n + 255) / 256);
    long long s = pairs / tiles;
    const int k_blocks = (k + kBlockK - 1) / kBlockK;
    if (s > 8) s = 8;
    if (s > k_blocks) s = k_blocks;
    return s < 1 ? 1 : (int)s;
}

// Y [m][n] = A^T B with A [k][m] and B [k][n] (the reduction index outermost in both), no bias: one launch.
// splits > 1: nothing is written to Y; partial [splits][m][n] receives the fp32 sums of each range of the reduction.
elsa_status launch_linear_tc_pair_tn(const uint16_t* A, const uint16_t* B, int m, int n, int k, elsa_dtype dtype,
                                     uint16_t* Y, int splits, float* partial, uint32_t* dev_status, cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    PairJob job;
    job.X = A; job.Wd = B; job.bias = nullptr; job.Y = Y;
    job.rows = m; job.in = k; job.out = n;
    job.splits = splits < 1 ? 1 : splits;
    job.partial = partial;
    return dtype == ELSA_BF16 ? launch_group<true, kFormTn, 1>(&job, 1, dtype, dev_status, stream, dev)
                              : launch_group<false, kFormTn, 1>(&job, 1, dtype, dev_status, stream, dev);
}

// INT8 form (one layer per launch): X and Wd hold signed 8-bit integers, Y is 16-bit.
elsa_status launch_linear_tc_pair_i8(const int8_t* X, int rows, const int8_t* Wd, const float* w_scale, float x_scale,
                                     const uint16_t* bias, int out, int in, elsa_dtype dtype, uint16_t* Y,
                                     uint32_t* dev_status, cudaStream_t stream)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    PairJob job;
    job.X = (const uint16_t*)X; job.Wd = (const uint16_t*)Wd; job.bias = bias; job.Y = Y;
    job.rows = rows; job.in = in; job.out = out;
    job.w_scale = w_scale; job.x_scale = x_scale;
    return dtype == ELSA_BF16 ? launch_group<true, kFormInt8, 1>(&job, 1, dtype, dev_status, stream, dev)
                              : launch_group<false, kFormInt8, 1>(&job, 1, dtype, dev_status, stream, dev);
}

elsa_status launch_linear_tc_pair(const uint16_t* X, int rows, const uint16_t* Wd, const uint16_t* bias, int out,
                                  int in, elsa_dtype dtype, uint16_t* Y, uint32_t* dev_status, cudaStream_t stream)
{
    PairJob job;
    job.X = X; job.Wd = Wd; job.bias = bias; job.Y = Y;
    job.rows = rows; job.in = in; job.out = out;
    job.w_scale = nullptr; job.x_scale = 0.f;
    return launch_linear_tc_pair_group(&job, 1, dtype, dev_status, stream);
}

}  // namespace elsa
