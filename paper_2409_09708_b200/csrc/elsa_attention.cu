// Multi-head self-attention of the ViT block between the pruned qkv and proj linears (ELSA, Sec. 3: the paper
// prunes the four linear modules and leaves the attention products dense; Sec. 4.2 measures whole models).
//     a[img, :, h] = softmax(q k^T / sqrt d) v      per image and head, over the keys of the same image
// with q, k, v the head's 64 columns in the three thirds of qkv [images * tokens][3 * dim].
//
// Work item = (128 query rows, head, image); tokens <= 256, head dimension 64 (the ViT / DeiT shapes) or 32 (Swin).
// An "image" is whatever set of consecutive rows attends within itself: for Swin, one window of the rolled grid, with
// an additive fp32 table per head on the scores (relative-position bias) and a second one per window position
// (the seam mask of shifted windows); the biased form is an instantiation of its own.  Both
// products run on tcgen05 with everything between them kept on chip:
//   1. TMA brings the Q tile, all K rows and all V rows of the head into shared memory (128-byte swizzle; a 3-D
//      tensor map [image][token][column] zero-fills the rows past the image's last token).
//   2. S = Q K^T: four MMAs (K = 16 each) into Tk = tokens rounded up to 16 fp32 columns of tensor memory.
//   3. Four warps, one query row per lane: row maximum over the real keys, p = 2^((s - max) * log2(e) / 8), row
//      sum in fp32, p rounded to the 16-bit type and written back into tensor memory as the A operand of the
//      second product, two keys per column, over the low half of the columns S occupied.
//   4. O = P V: Tk / 16 MMAs with A from tensor memory and V as it lies in memory (keys outermost: MN-major
//      descriptor) into 64 columns of the part of S that is dead by then.
//   5. The same four warps read O, divide by the row sum, round once and store each row's 128 bytes.
// Persistent: one CTA per SM walks the items with the stride of the grid, with several items in flight: two for up
// to 256 keys, four for up to 128 (Swin's windows), each with its own shared-memory stage (Q, K, V), its own share
// of tensor memory (256 or 128 columns) and its own group of four softmax warps: item n uses stage, share and group
// n % 2 (n % 4).  The producer warp loads ahead as stages come free (Q and K of a stage after the scores of its
// previous item, V after that item's second product); the MMA warp issues S of item n, then P V of the
// oldest item whose probabilities are due, so one group's softmax runs under the others' products and epilogues.
// Every wait is bounded as in the GEMM kernels.
#include <atomic>
#include <mutex>

#include "elsa_tc_common.cuh"

namespace elsa {
namespace {

constexpr int kMaxHeadDim = 64;
constexpr int kQRows = 128;          // query rows per item = TMEM lanes
constexpr int kMaxTokens = 256;
constexpr int kTmemCols = 512;
constexpr int kGroupWarps = 4;       // softmax warps per group, one per TMEM lane quarter
constexpr int kQBytes = kQRows * kMaxHeadDim * 2;          // the shared-memory slots are laid out for head dimension 64

// kBufs items in flight per CTA: 2 for up to 256 keys (256 tensor-memory columns each), 4 for up to 128 keys (the
// windows of Swin), where an item's on-chip chain is short and only more of them in flight fill the SM.
template <int kBufs>
struct Shape {
    static constexpr int kBufCols = kTmemCols / kBufs;
    static constexpr int kThreads = (2 + kBufs * kGroupWarps) * 32;
    static constexpr int kKvBytes = (kBufs == 2 ? 256 : 128) * kMaxHeadDim * 2;
    static constexpr int kStageBytes = kQBytes + 2 * kKvBytes;
    static constexpr int kSmemBytes = kBufs * kStageBytes + 1024 /* alignment */ + 512 /* barriers */;
    static constexpr int kUnit = kBufs == 2 ? 32 : 16;      // score columns a softmax warp handles at a time (registers)
};

struct AttnParams {
    CUtensorMap map_q;    // box 64 columns x 128 tokens x 1 image
    CUtensorMap map_kv;   // box 64 columns x Tk tokens x 1 image
    uint16_t* out;        // [images * tokens][dim]
    int tokens, tk, dim;
    int m_tiles, heads, items;   // items = images * heads * m_tiles, query tile fastest
    int o_col;            // first column of O inside an item's half of tensor memory
    uint32_t idesc_s, idesc_o;
    uint32_t* dev_status;
    // biased form: scores get bias[head][row][key] + mask[image % n_masks][row][key] (fp32, rows of bias_pitch floats)
    const float* bias;
    const float* mask;    // or NULL
    int n_masks, bias_pitch;
};

// MN-major tile of rows of 64 bytes (32 16-bit values along N per reduction index) with the 64-byte swizzle: 8
// reduction rows form a 512-byte group.
__device__ __forceinline__ uint64_t smem_desc_mn_major_sw64(uint32_t addr, uint32_t block_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((block_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(512 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)4 << 61;
    return d;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

// D[tmem] (+)= A[tmem] * B[smem]: A's 16-bit values two per column, lane = row.  Predicated as the other forms.
__device__ __forceinline__ void umma_f16_ts_if(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
        : "memory");
}

__device__ __forceinline__ void tmem_st_32x32b_x8(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"r"(taddr), "r"(r[0]),
                 "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

template <bool kBf16, int kD, bool kBias, int kBufs>
__global__ void __launch_bounds__(Shape<kBufs>::kThreads, 1) attention_kernel(const __grid_constant__ AttnParams p)
{
    static_assert(kD == 64 || kD == 32, "head dimension");
    static_assert(kBufs == 2 || kBufs == 4, "items in flight");
    constexpr int kBufCols = Shape<kBufs>::kBufCols, kStageBytes = Shape<kBufs>::kStageBytes, kKvBytesMax = Shape<kBufs>::kKvBytes;
    constexpr int U = Shape<kBufs>::kUnit;
    constexpr int kLag = kBufs - 1;                   // P V of item n - kLag is issued after S of item n
    constexpr int kHeadDim = kD;
    constexpr int kItemQBytes = kQRows * kD * 2;      // bytes TMA delivers for the Q tile; K and V: tk * kD * 2
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t bars = smem_base + kBufs * kStageBytes;
    // per buffer b: +0 qk_full, +8 v_full, +16 qk_empty, +24 s_full, +32 p_full, +40 o_full, +48 tmem_empty, +56 v_empty
    auto bar = [&](int which, int b) { return bars + (uint32_t)(64 * b + 8 * which); };
    enum { kQkFull = 0, kVFull, kQkEmpty, kSFull, kPFull, kOFull, kTmemEmpty, kVEmpty };
    const uint32_t tmem_holder_addr = bars + 64 * kBufs;
    uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem_raw + (tmem_holder_addr - smem_u32(smem_raw)));
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_raw + (bars + 64 * kBufs + 8 - smem_u32(smem_raw)));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int first = blockIdx.x, stride = gridDim.x;
    const int n_items = first < p.items ? (p.items - first + stride - 1) / stride : 0;   // items of this CTA

    if (warp == 1) {
        if (lane == 0) {
            for (int b = 0; b < kBufs; ++b) {
                mbar_init(bar(kQkFull, b), 1);
                mbar_init(bar(kVFull, b), 1);
                mbar_init(bar(kQkEmpty, b), 1);
                mbar_init(bar(kVEmpty, b), 1);
                mbar_init(bar(kSFull, b), 1);
                mbar_init(bar(kPFull, b), kGroupWarps);
                mbar_init(bar(kOFull, b), 1);
                mbar_init(bar(kTmemEmpty, b), kGroupWarps);
            }
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        __syncwarp();
        tmem_alloc(tmem_holder_addr, kTmemCols);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    pdl_wait_for_predecessors();
    pdl_release_successors();

    if (warp == 0) {
        // ------------------------------------------------ TMA producer
        const bool elected = elect_one();
        bool ok = true;
        // Q and K of a stage are free as soon as the scores of its previous item are complete, V only after that item's
        // second product.  The loop asks for Q and K of item n, then for V of item n - 1: the order in which the MMA
        // warp frees them (S of item n - kBufs, then P V of item n - 1 - kBufs), so the next item's Q and K arrive under
        // the softmax, off the chain of the buffer, and no wait holds back a load whose stage is free already.
        for (int n = 0; ok && n <= n_items; ++n) {
            if (n < n_items) {
                const int b = n % kBufs;
                const uint32_t ph = (uint32_t)((n / kBufs) & 1);
                ok = mbar_wait(bar(kQkEmpty, b), ph ^ 1u, abort_flag, p.dev_status, 20);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                const int item = first + n * stride;
                const int mt = item % p.m_tiles, head = (item / p.m_tiles) % p.heads, img = item / (p.m_tiles * p.heads);
                const uint32_t q_smem = smem_base + (uint32_t)(b * kStageBytes);
                if (elected) {
                    mbar_arrive_expect_tx(bar(kQkFull, b), (uint32_t)(kItemQBytes + p.tk * kHeadDim * 2));
                    tma_load_3d(q_smem, &p.map_q, bar(kQkFull, b), head * kHeadDim, mt * kQRows, img);
                    tma_load_3d(q_smem + kQBytes, &p.map_kv, bar(kQkFull, b), p.dim + head * kHeadDim, 0, img);
                }
                __syncwarp();
            }
            if (n >= 1) {
                const int m = n - 1, b = m % kBufs;
                const uint32_t ph = (uint32_t)((m / kBufs) & 1);
                ok = mbar_wait(bar(kVEmpty, b), ph ^ 1u, abort_flag, p.dev_status, 27);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                const int item = first + m * stride;
                const int head = (item / p.m_tiles) % p.heads, img = item / (p.m_tiles * p.heads);
                const uint32_t q_smem = smem_base + (uint32_t)(b * kStageBytes);
                if (elected) {
                    mbar_arrive_expect_tx(bar(kVFull, b), (uint32_t)(p.tk * kHeadDim * 2));
                    tma_load_3d(q_smem + kQBytes + kKvBytesMax, &p.map_kv, bar(kVFull, b), 2 * p.dim + head * kHeadDim, 0, img);
                }
                __syncwarp();
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issuer: S of item n, then P V of item n - 1
        const uint32_t elected = elect_one() ? 1u : 0u;
        const uint32_t tmem_u = __reduce_or_sync(0xFFFFFFFFu, tmem_base);
        const int steps = p.tk / 16;
        bool ok = true;
        for (int n = 0; ok && n < n_items + kLag; ++n) {
            if (n < n_items) {
                const int b = n % kBufs;
                const uint32_t ph = (uint32_t)((n / kBufs) & 1);
                ok = mbar_wait(bar(kTmemEmpty, b), ph ^ 1u, abort_flag, p.dev_status, 21);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                ok = mbar_wait(bar(kQkFull, b), ph, abort_flag, p.dev_status, 22);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t q_smem = smem_base + (uint32_t)(b * kStageBytes);
                const uint64_t a_desc = kD == 64 ? smem_desc_k_major_sw128(q_smem) : smem_desc_k_major_sw64(q_smem);
                const uint64_t b_desc = kD == 64 ? smem_desc_k_major_sw128(q_smem + kQBytes) : smem_desc_k_major_sw64(q_smem + kQBytes);
#pragma unroll
                for (int k = 0; k < kHeadDim / 16; ++k)
                    umma_f16_if(tmem_u + (uint32_t)(b * kBufCols), a_desc + (uint64_t)(2 * k), b_desc + (uint64_t)(2 * k), p.idesc_s,
                                (uint32_t)(k != 0), elected);
                umma_commit_if(bar(kSFull, b), elected);
                umma_commit_if(bar(kQkEmpty, b), elected);     // Q and K of the stage have been read
            }
            if (n >= kLag) {
                const int m = n - kLag, b = m % kBufs;
                const uint32_t ph = (uint32_t)((m / kBufs) & 1);
                ok = mbar_wait(bar(kVFull, b), ph, abort_flag, p.dev_status, 23);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                ok = mbar_wait(bar(kPFull, b), ph, abort_flag, p.dev_status, 24);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_buf = tmem_u + (uint32_t)(b * kBufCols);
                const uint32_t v_smem = smem_base + (uint32_t)(b * kStageBytes + kQBytes + kKvBytesMax);
                const uint64_t v_desc = kD == 64 ? smem_desc_mn_major_sw128(v_smem, (uint32_t)(p.tk * kHeadDim * 2))
                                                 : smem_desc_mn_major_sw64(v_smem, (uint32_t)(p.tk * kHeadDim * 2));
                // 16 keys of kD * 2 bytes per MMA
                for (int k = 0; k < steps; ++k)
                    umma_f16_ts_if(t_buf + (uint32_t)p.o_col, t_buf + (uint32_t)(8 * k), v_desc + (uint64_t)(k * (16 * kD * 2 >> 4)),
                                   p.idesc_o, (uint32_t)(k != 0), elected);
                umma_commit_if(bar(kOFull, b), elected);
                umma_commit_if(bar(kVEmpty, b), elected);      // V of the stage has been read
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------ softmax and output: group g takes the items n = g, g + 2, ...
        const int g = (warp - 2) / kGroupWarps;
        const int quarter = warp & 3;                                  // the TMEM lanes this warp may touch
        const float scale = (kD == 64 ? 0.125f : 0.17677669529663687f) * 1.4426950408889634f;   // log2(e) / sqrt(kD)
        bool ok = true;
        for (int n = g; ok && n < n_items; n += kBufs) {
            const uint32_t ph = (uint32_t)((n / kBufs) & 1);
            const int item = first + n * stride;
            const int mt = item % p.m_tiles, head = (item / p.m_tiles) % p.heads, img = item / (p.m_tiles * p.heads);
            const int row = mt * kQRows + quarter * 32 + lane;         // token index inside the image
            const uint32_t t_lane = tmem_base + (uint32_t)(g * kBufCols) + ((uint32_t)(quarter * 32) << 16);
            float sum = 0.f;
            // biased form: what is exponentiated is s * scale + (bias + mask) * log2(e); the tables' rows of this lane
            const float* brow = nullptr;
            const float* mrow = nullptr;
            if constexpr (kBias) {
                if (row < p.tokens) {
                    brow = p.bias + ((size_t)head * p.tokens + row) * (size_t)p.bias_pitch;
                    if (p.mask != nullptr) mrow = p.mask + ((size_t)(img % p.n_masks) * p.tokens + row) * (size_t)p.bias_pitch;
                }
            }
            // (bias + mask) * log2(e) for `count` columns from col0 (multiples of 4; rows of the tables are 16-byte
            // aligned and padded to bias_pitch, so whole float4 loads stay inside a row); zeros without tables
            auto load_bias = [&](float* bb, int col0, int count) {
#pragma unroll
                for (int v = 0; v < 8; ++v) {
                    if (4 * v >= count) break;
                    float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (brow != nullptr && col0 + 4 * v < p.bias_pitch) {
                        b4 = __ldg(reinterpret_cast<const float4*>(brow + col0) + v);
                        if (mrow != nullptr) {
                            const float4 m4 = __ldg(reinterpret_cast<const float4*>(mrow + col0) + v);
                            b4.x += m4.x; b4.y += m4.y; b4.z += m4.z; b4.w += m4.w;
                        }
                    }
                    bb[4 * v] = b4.x * 1.4426950408889634f; bb[4 * v + 1] = b4.y * 1.4426950408889634f;
                    bb[4 * v + 2] = b4.z * 1.4426950408889634f; bb[4 * v + 3] = b4.w * 1.4426950408889634f;
                }
            };
            // The bias table's values of one unit, as loaded (no arithmetic on them here, so a request stays in flight
            // until the values are used): the first unit is asked for before the scores are waited for, every other
            // one while the unit before it is worked on, which takes most of the L2 latency out of the item's chain.
            // The mask (shifted windows only) is read where it is used: a second array across the wait would spill.
            constexpr int kReq = kBias ? Shape<kBufs>::kUnit : 1;
            float bq[kReq];
            auto request = [&](int col0) {
#pragma unroll
                for (int v = 0; v < kReq / 4; ++v) {
                    float4 b4 = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (brow != nullptr && col0 + 4 * v < p.bias_pitch) b4 = __ldg(reinterpret_cast<const float4*>(brow + col0) + v);
                    bq[4 * v] = b4.x; bq[4 * v + 1] = b4.y; bq[4 * v + 2] = b4.z; bq[4 * v + 3] = b4.w;
                }
            };
            if constexpr (kBias) request(0);
            ok = mbar_wait(bar(kSFull, g), ph, abort_flag, p.dev_status, 25);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            {
                // Tensor-memory reads are waited for all at once, so the loads of a pass are issued in batches: the
                // row maximum from two units per round trip, the second pass with the next unit in flight while
                // the current one is exponentiated.  A unit is U = 32 score columns (16 with four items in flight).
                auto ld_unit = [&](uint32_t taddr, uint32_t (&r)[U]) {
                    if constexpr (U == 32) tmem_ld_32x32b_x32(taddr, r);
                    else tmem_ld_32x32b_x16(taddr, r);
                };
                const int units = p.tk / U;                      // whole units
                const bool tail = U == 32 && (p.tk & 31) != 0;   // plus one chunk of 16
                float m = -INFINITY;
                if constexpr (kBias) {
                    // first pass of the biased form: t = s * scale + (bias + mask) * log2(e) replaces s in tensor memory,
                    // so the tables are read once
                    for (int u = 0; u < units; ++u) {
                        uint32_t r[U];
                        float bb[U];
                        ld_unit(t_lane + (uint32_t)(U * u), r);
#pragma unroll
                        for (int v = 0; v < U / 4; ++v) {
                            float4 m4 = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (mrow != nullptr && U * u + 4 * v < p.bias_pitch) m4 = __ldg(reinterpret_cast<const float4*>(mrow + U * u) + v);
                            bb[4 * v] = (bq[4 * v] + m4.x) * 1.4426950408889634f;
                            bb[4 * v + 1] = (bq[4 * v + 1] + m4.y) * 1.4426950408889634f;
                            bb[4 * v + 2] = (bq[4 * v + 2] + m4.z) * 1.4426950408889634f;
                            bb[4 * v + 3] = (bq[4 * v + 3] + m4.w) * 1.4426950408889634f;
                        }
                        if (u + 1 < units) request(U * (u + 1));
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < U; ++j) {
                            const float t = fmaf(__uint_as_float(r[j]), scale, bb[j]);
                            r[j] = __float_as_uint(t);
                            if (U * u + j < p.tokens) m = fmaxf(m, t);
                        }
#pragma unroll
                        for (int h = 0; h < U / 16; ++h) {
                            uint32_t part[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) part[j] = r[16 * h + j];
                            tmem_st_32x32b_x16(t_lane + (uint32_t)(U * u + 16 * h), part);
                        }
                    }
                    if (tail) {
                        uint32_t r[16];
                        float bb[16];
                        tmem_ld_32x32b_x16(t_lane + (uint32_t)(U * units), r);
                        load_bias(bb, U * units, 16);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float t = fmaf(__uint_as_float(r[j]), scale, bb[j]);
                            r[j] = __float_as_uint(t);
                            if (U * units + j < p.tokens) m = fmaxf(m, t);
                        }
                        tmem_st_32x32b_x16(t_lane + (uint32_t)(U * units), r);
                    }
                    tmem_wait_st();
                } else {
                    for (int u0 = 0; u0 < units; u0 += 2) {
                        uint32_t r[2][U];
#pragma unroll
                        for (int i = 0; i < 2; ++i)
                            if (u0 + i < units) ld_unit(t_lane + (uint32_t)(U * (u0 + i)), r[i]);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 2; ++i)
                            if (u0 + i < units) {
                                if (U * (u0 + i) + U <= p.tokens) {       // a unit of real keys only: no per-column test
                                    float m0 = m, m1 = -INFINITY;
#pragma unroll
                                    for (int j = 0; j < U; j += 2) {
                                        m0 = fmaxf(m0, __uint_as_float(r[i][j]));
                                        m1 = fmaxf(m1, __uint_as_float(r[i][j + 1]));
                                    }
                                    m = fmaxf(m0, m1);
                                } else {
#pragma unroll
                                    for (int j = 0; j < U; ++j)
                                        if (U * (u0 + i) + j < p.tokens) m = fmaxf(m, __uint_as_float(r[i][j]));
                                }
                            }
                    }
                    if (tail) {
                        uint32_t r[16];
                        tmem_ld_32x32b_x16(t_lane + (uint32_t)(U * units), r);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (U * units + j < p.tokens) m = fmaxf(m, __uint_as_float(r[j]));
                    }
                }
                // p = 2^(s * scale - m * scale) for 16 columns starting at col0: eight packed pairs
                const float m_scaled = kBias ? m : m * scale;      // the biased maximum is in the exponent's domain already
                float sum1 = 0.f;
                auto exp16 = [&](const uint32_t* r, int col0, uint32_t (&w)[8]) {
                    const bool all_real = col0 + 16 <= p.tokens;
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        float e0, e1;
                        const float a0 = kBias ? __uint_as_float(r[2 * j]) - m_scaled : fmaf(__uint_as_float(r[2 * j]), scale, -m_scaled);
                        const float a1 = kBias ? __uint_as_float(r[2 * j + 1]) - m_scaled
                                               : fmaf(__uint_as_float(r[2 * j + 1]), scale, -m_scaled);
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(a0));
                        asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(a1));
                        if (!all_real) {                                  // padded keys take no part
                            if (col0 + 2 * j >= p.tokens) e0 = 0.f;
                            if (col0 + 2 * j + 1 >= p.tokens) e1 = 0.f;
                        }
                        sum += e0;
                        sum1 += e1;
                        w[j] = pack2<kBf16>(e0, e1);
                    }
                };
                // P's columns of a unit lie over S columns of units that have been read already
                auto unit = [&](const uint32_t (&r)[U], int u) {
#pragma unroll
                    for (int h = 0; h < U / 16; ++h) {
                        uint32_t w[8];
                        exp16(&r[16 * h], U * u + 16 * h, w);
                        tmem_st_32x32b_x8(t_lane + (uint32_t)(U / 2 * u + 8 * h), w);
                    }
                };
                uint32_t ra[U], rb[U];
                if (units > 0) ld_unit(t_lane, ra);
                for (int u = 0; u < units; u += 2) {
                    tmem_wait_ld();
                    if (u + 1 < units) ld_unit(t_lane + (uint32_t)(U * (u + 1)), rb);
                    unit(ra, u);
                    if (u + 1 < units) {
                        tmem_wait_ld();
                        if (u + 2 < units) ld_unit(t_lane + (uint32_t)(U * (u + 2)), ra);
                        unit(rb, u + 1);
                    }
                }
                if (tail) {
                    uint32_t r[16], w[8];
                    tmem_ld_32x32b_x16(t_lane + (uint32_t)(U * units), r);
                    tmem_wait_ld();
                    exp16(r, U * units, w);
                    tmem_st_32x32b_x8(t_lane + (uint32_t)(U / 2 * units), w);
                }
                sum += sum1;
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kPFull, g));
            ok = mbar_wait(bar(kOFull, g), ph, abort_flag, p.dev_status, 26);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            const float inv = 1.0f / sum;
            uint32_t w[kD / 16][8];                                    // the row's kD outputs, packed
#pragma unroll
            for (int half = 0; half < kD / 32; ++half) {
                uint32_t o[2][16];
                tmem_ld_32x32b_x16(t_lane + (uint32_t)(p.o_col + 32 * half), o[0]);
                tmem_ld_32x32b_x16(t_lane + (uint32_t)(p.o_col + 32 * half + 16), o[1]);
                tmem_wait_ld();
#pragma unroll
                for (int q = 0; q < 2; ++q)
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        w[2 * half + q][j] = pack2<kBf16>(__uint_as_float(o[q][2 * j]) * inv, __uint_as_float(o[q][2 * j + 1]) * inv);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kTmemEmpty, g));            // the half may take the S of item n + 2
            if (row < p.tokens) {
                uint4* dst = reinterpret_cast<uint4*>(p.out + ((size_t)img * p.tokens + row) * (size_t)p.dim + head * kHeadDim);
#pragma unroll
                for (int q = 0; q < kD / 16; ++q) {
                    dst[2 * q] = make_uint4(w[q][0], w[q][1], w[q][2], w[q][3]);
                    dst[2 * q + 1] = make_uint4(w[q][4], w[q][5], w[q][6], w[q][7]);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

elsa_status make_map_qkv(CUtensorMap* map, const void* qkv, int images, int tokens, int dim, int head_dim, uint32_t box_rows,
                         const char* what)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(ELSA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {(cuuint64_t)(3 * dim), (cuuint64_t)tokens, (cuuint64_t)images};
    cuuint64_t strides[2] = {(cuuint64_t)(3 * dim) * 2, (cuuint64_t)tokens * (cuuint64_t)(3 * dim) * 2};
    cuuint32_t box[3] = {(cuuint32_t)head_dim, box_rows, 1};
    cuuint32_t elem[3] = {1, 1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(qkv), dims, strides, box, elem,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, head_dim == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
                     CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ELSA_ERR_CUDA, "tensor map for %s rejected (CUresult %d)", what, (int)rc);
    return ELSA_OK;
}

template <bool kBf16, int kD, bool kBias, int kBufs>
elsa_status launch(const AttnParams& p, int images, int heads, cudaStream_t stream, const DeviceInfo& dev)
{
    constexpr int kSmemBytes = Shape<kBufs>::kSmemBytes, kThreads = Shape<kBufs>::kThreads;
    auto kernel = attention_kernel<kBf16, kD, kBias, kBufs>;
    static std::atomic<bool> attr_set[64];
    const int slot = dev.device & 63;
    if (!attr_set[slot].load(std::memory_order_acquire)) {
        if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes) != cudaSuccess) {
            cudaError_t e = cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(e));
        }
        attr_set[slot].store(true, std::memory_order_release);
    }
    (void)images;
    (void)heads;
    const dim3 grid((unsigned)(p.items < dev.sm_count ? p.items : dev.sm_count));   // one persistent CTA per SM
    ProfileScope scope(ELSA_KERNEL_ATTENTION, stream);
    cudaError_t e = launch_pdl(kernel, grid, dim3(kThreads), (size_t)kSmemBytes, stream, 1, p);
    if (e != cudaSuccess) return fail(ELSA_ERR_CUDA, "attention launch: %s", cudaGetErrorString(e));
    return launched("attention");
}

}  // namespace

bool attention_suits(int tokens, int heads, int dim)
{
    return tokens >= 1 && tokens <= kMaxTokens && heads >= 1 && (dim == heads * 64 || dim == heads * 32);
}

elsa_status launch_attention(const uint16_t* qkv, int images, int tokens, int heads, int dim, elsa_dtype dtype,
                             uint16_t* out, uint32_t* dev_status, cudaStream_t stream, const float* bias, const float* mask,
                             int n_masks, int bias_pitch)
{
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    if (!attention_suits(tokens, heads, dim))
        return fail(ELSA_ERR_SHAPE, "attention needs 1..%d tokens per image and a head dimension of 32 or 64 (tokens=%d, heads=%d, dim=%d)",
                    kMaxTokens, tokens, heads, dim);
    const int head_dim = dim / heads;
    if (bias == nullptr && mask != nullptr) return fail(ELSA_ERR_NULL, "a mask table needs a bias table");
    if (bias != nullptr && (bias_pitch < tokens || bias_pitch % 4 != 0 || (mask != nullptr && n_masks < 1)))
        return fail(ELSA_ERR_SHAPE, "bias_pitch=%d must be a multiple of 4 and at least tokens=%d, n_masks=%d at least 1", bias_pitch,
                    tokens, n_masks);
    if (bias != nullptr && ((((uintptr_t)bias) & 15u) != 0 || (((uintptr_t)mask) & 15u) != 0))
        return fail(ELSA_ERR_ALIGN, "the bias and mask tables must be 16-byte aligned");
    if ((long long)images * heads * ((tokens + kQRows - 1) / kQRows) > 0x7fffffffLL)
        return fail(ELSA_ERR_SHAPE, "images * heads does not fit an int");
    AttnParams p;
    p.out = out;
    p.tokens = tokens;
    p.tk = (tokens + 15) / 16 * 16;
    p.dim = dim;
    p.m_tiles = (tokens + kQRows - 1) / kQRows;
    p.heads = heads;
    p.items = images * heads * p.m_tiles;
    // O (head_dim columns) over the part of S that P does not cover (P: tk / 2 columns from 0; S is dead by then)
    p.o_col = (p.tk / 2 + 31) / 32 * 32;
    const uint32_t fmt = dtype == ELSA_BF16 ? 1u : 0u;
    p.idesc_s = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(p.tk >> 3) << 17) | ((uint32_t)(kQRows >> 4) << 24);
    p.idesc_o = (1u << 4) | (fmt << 7) | (fmt << 10) | (1u << 16) | ((uint32_t)(head_dim >> 3) << 17) | ((uint32_t)(kQRows >> 4) << 24);
    p.dev_status = dev_status;
    p.bias = bias; p.mask = mask; p.n_masks = n_masks > 0 ? n_masks : 1; p.bias_pitch = bias_pitch;
    if ((st = make_map_qkv(&p.map_q, qkv, images, tokens, dim, head_dim, kQRows, "q")) != ELSA_OK) return st;
    if ((st = make_map_qkv(&p.map_kv, qkv, images, tokens, dim, head_dim, (uint32_t)p.tk, "k, v")) != ELSA_OK) return st;
    const bool bf = dtype == ELSA_BF16, biased = bias != nullptr;
    const bool four = p.tk <= 128;       // short chains: four items in flight per CTA
#define ELSA_ATTN(D, B, N) (bf ? launch<true, D, B, N>(p, images, heads, stream, dev) : launch<false, D, B, N>(p, images, heads, stream, dev))
    if (head_dim == 64) {
        if (biased) return four ? ELSA_ATTN(64, true, 4) : ELSA_ATTN(64, true, 2);
        return four ? ELSA_ATTN(64, false, 4) : ELSA_ATTN(64, false, 2);
    }
    if (biased) return four ? ELSA_ATTN(32, true, 4) : ELSA_ATTN(32, true, 2);
    return four ? ELSA_ATTN(32, false, 4) : ELSA_ATTN(32, false, 2);
#undef ELSA_ATTN
}

}  // namespace elsa
