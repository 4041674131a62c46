// N:M projection of a weight matrix and its compressed form, and the inverse.
//
// elsa_nm_compress: Sec. 3.1 / Eq. 1 of the ELSA paper with magnitude saliency (keep the N largest
// |w| of each group of M consecutive weights), written in the compressed form of Sec. 1 / Sec. 2
// (kept values + one log2(M)-bit index each).  Both kernels are plain streaming kernels: one
// 16-byte load per group of eight, integer compares, coalesced word stores.

#include "elsa_pack_device.cuh"

namespace elsa {
namespace {

template <int M>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
nm_compress_kernel(const uint16_t* __restrict__ W, int out, int in, int N, uint16_t* __restrict__ vals,
                   uint32_t* __restrict__ idx, int segs_per_row, int words_per_row)
{
    __shared__ uint32_t words[kWarpsPerBlock][kMaxIndexWordsPerSegment];
    __shared__ CompactEntry table[M == 16 ? 1 : (1 << M)];
    if constexpr (M != 16) {
        build_compact_table<M>(table);
        __syncthreads();
    }
    pdl_wait_for_predecessors();
    pdl_release_successors();
    // warps walk the segments with the stride of the grid (whole warps leave together; no block-wide barrier follows)
    const long long total = (long long)out * segs_per_row;
    for (long long seg_id = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5); seg_id < total;
         seg_id += (long long)gridDim.x * kWarpsPerBlock) {
        if constexpr (M == 16) compress_segment<M>(W, in, N, vals, idx, segs_per_row, words_per_row, seg_id, words);
        else compress_segment_fast<M>(W, in, N, vals, idx, segs_per_row, seg_id, words, table);
    }
}

template <int M>
__global__ void __launch_bounds__(256)
nm_unpack_kernel(const uint16_t* __restrict__ vals, const uint32_t* __restrict__ idx, int out, int in,
                 int N, uint16_t* __restrict__ Wm, int words_per_row)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (gid >= (long long)out * (in / M)) return;
    unpack_group<M>(vals, idx, in, N, Wm, words_per_row, gid);
}

// All requested levels N:M of one weight from a single read of it (the ranks do not depend on N).
template <int M>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
nm_compress_levels_kernel(const uint16_t* __restrict__ W, int out, int in, const LevelTable t, int segs_per_row)
{
    __shared__ uint32_t words[kWarpsPerBlock][kMaxIndexWordsPerSegment];
    const long long seg_id = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (seg_id >= (long long)out * segs_per_row) return;
    compress_segment_levels<M>(W, in, t.n, t.N, t.vals, t.idx, segs_per_row, seg_id, words);
}

// Dense weight projected onto level N:M, still dense (pruned positions +0.0).
template <int M>
__global__ void __launch_bounds__(256)
nm_mask_kernel(const uint16_t* __restrict__ W, long long groups, int N, uint16_t* __restrict__ Wm)
{
    const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    pdl_wait_for_predecessors();
    pdl_release_successors();
    if (gid >= groups) return;
    mask_group<M>(W, N, Wm, gid);
}

// ---- batched forms: one launch over a table of weights.  A unit is a warp segment (compress) or a
// thread (weight-image kernels); every block looks its first unit up in the table's prefix sums.

__device__ __forceinline__ int find_item(const BatchTable& t, long long unit)
{
    int lo = 0, hi = t.n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (t.item[mid].first_unit <= unit) lo = mid; else hi = mid - 1;
    }
    return lo;
}

// Groups of 16 take the general path; kept out of line so that its registers do not count against the
// fast path of the batched kernel.
__device__ __noinline__ void compress_segment16_call(const uint16_t* W, int in, int N, uint16_t* vals, uint32_t* idx,
                                                     int segs_per_row, int words_per_row, long long seg_id,
                                                     uint32_t (*words)[kMaxIndexWordsPerSegment])
{
    compress_segment<16>(W, in, N, vals, idx, segs_per_row, words_per_row, seg_id, words);
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32, 4)
nm_compress_batch_kernel(const __grid_constant__ BatchTable t)
{
    __shared__ uint32_t words[kWarpsPerBlock][kMaxIndexWordsPerSegment];
    __shared__ CompactEntry table8[256];
    __shared__ CompactEntry table4[16];
    build_compact_table<8>(table8);
    build_compact_table<4>(table4);
    __syncthreads();
    pdl_wait_for_predecessors();
    pdl_release_successors();
    // A block owns a contiguous range of units and its warps walk it side by side; the table is searched
    // once per block and stepped through afterwards (a search per unit costs several dependent reads of
    // kernel-parameter memory, more than the unit's own work).  The fields of the current weight live in
    // registers: reading them from the parameter table with a computed index for every unit kept the
    // pipe that serves such reads busier than any other.
    const long long per_block = (t.total_units + gridDim.x - 1) / gridDim.x;
    const long long begin = (long long)blockIdx.x * per_block;
    const long long end = begin + per_block < t.total_units ? begin + per_block : t.total_units;
    if (begin >= end) return;
    int cur = find_item(t, begin);
    long long cur_end;
    const uint16_t* W; uint16_t* vals; uint32_t* idx;
    long long first_unit;
    int in, N, M, segs_per_row, wpr;
    auto load_item = [&]() {
        const BatchItem& it = t.item[cur];
        cur_end = cur + 1 < t.n ? t.item[cur + 1].first_unit : t.total_units;
        W = (const uint16_t*)it.src; vals = (uint16_t*)it.dst; idx = (uint32_t*)it.dst2;
        first_unit = it.first_unit;
        in = it.in; N = it.N; M = it.M; segs_per_row = it.aux; wpr = it.wpr;
    };
    load_item();
    // Software pipeline: the 16 bytes of the next unit are requested before the current one is worked on.  With
    // one load per warp in flight the kernel moved exactly (resident warps x 512 bytes) per memory latency.
    const int lane = threadIdx.x & 31;
    uint32_t nr[4] = {0u, 0u, 0u, 0u};
    int n_o = 0, n_seg = 0;
    auto request = [&](long long unit) {          // `unit` belongs to the weight whose fields are loaded
        const uint32_t local = (uint32_t)(unit - first_unit);      // a weight has far fewer than 2^32 segments
        const uint32_t o = local / (uint32_t)segs_per_row;
        n_o = (int)o;
        n_seg = (int)(local - o * (uint32_t)segs_per_row);
        const int g = n_seg * 32 + lane;
        nr[0] = nr[1] = nr[2] = nr[3] = 0u;
        if (M == 8) {
            if (g < in / 8) { const uint4 v = *reinterpret_cast<const uint4*>(W + (size_t)n_o * in + (size_t)g * 8); nr[0] = v.x; nr[1] = v.y; nr[2] = v.z; nr[3] = v.w; }
        } else if (M == 4) {
            if (g < in / 4) { const uint2 v = *reinterpret_cast<const uint2*>(W + (size_t)n_o * in + (size_t)g * 4); nr[0] = v.x; nr[1] = v.y; }
        }
    };
    long long unit = begin + (threadIdx.x >> 5);
    while (unit < end) {
        if (unit >= cur_end) {
            while (unit >= (cur + 1 < t.n ? t.item[cur + 1].first_unit : t.total_units)) ++cur;
            load_item();
        }
        // this warp's units inside the current weight: its fields stay put, and the pipeline drains only
        // where the block's range crosses into the next weight
        const long long stop = cur_end < end ? cur_end : end;
        request(unit);
        for (; unit < stop; unit += kWarpsPerBlock) {
            const uint32_t r[4] = {nr[0], nr[1], nr[2], nr[3]};
            const int o = n_o, seg = n_seg;
            if (unit + kWarpsPerBlock < stop) request(unit + kWarpsPerBlock);
            // the levels of the ViT tables get the level as a compile-time constant
            if (M == 8) {
                switch (N) {
                case 1: compress_segment_fast_preloaded<8, 1>(r, in, 1, vals, idx, o, seg, words, table8); break;
                case 2: compress_segment_fast_preloaded<8, 2>(r, in, 2, vals, idx, o, seg, words, table8); break;
                case 4: compress_segment_fast_preloaded<8, 4>(r, in, 4, vals, idx, o, seg, words, table8); break;
                case 8: compress_segment_fast_preloaded<8, 8>(r, in, 8, vals, idx, o, seg, words, table8); break;
                default: compress_segment_fast_preloaded<8>(r, in, N, vals, idx, o, seg, words, table8); break;
                }
            } else if (M == 4) {
                switch (N) {
                case 1: compress_segment_fast_preloaded<4, 1>(r, in, 1, vals, idx, o, seg, words, table4); break;
                case 2: compress_segment_fast_preloaded<4, 2>(r, in, 2, vals, idx, o, seg, words, table4); break;
                case 4: compress_segment_fast_preloaded<4, 4>(r, in, 4, vals, idx, o, seg, words, table4); break;
                default: compress_segment_fast_preloaded<4>(r, in, N, vals, idx, o, seg, words, table4); break;
                }
            }
            else compress_segment16_call(W, in, N, vals, idx, segs_per_row, wpr, (long long)o * segs_per_row + seg, words);
        }
    }
}

__global__ void __launch_bounds__(256)
nm_image_batch_kernel(const __grid_constant__ BatchTable t)
{
    pdl_wait_for_predecessors();
    pdl_release_successors();
    // contiguous range of units per block, table searched once per block (see the compress kernel)
    const long long per_block = (t.total_units + gridDim.x - 1) / gridDim.x;
    const long long begin = (long long)blockIdx.x * per_block;
    const long long end = begin + per_block < t.total_units ? begin + per_block : t.total_units;
    if (begin >= end) return;
    int cur = find_item(t, begin);
    long long cur_end = cur + 1 < t.n ? t.item[cur + 1].first_unit : t.total_units;
    BatchItem it = t.item[cur];
    for (long long unit = begin + threadIdx.x; unit < end; unit += blockDim.x) {
        if (unit >= cur_end) {
            while (unit >= cur_end) {
                ++cur;
                cur_end = cur + 1 < t.n ? t.item[cur + 1].first_unit : t.total_units;
            }
            it = t.item[cur];
        }
        const long long local = unit - it.first_unit;
        const uint16_t* vals = (const uint16_t*)it.src;
        const uint32_t* idx = (const uint32_t*)it.src2;
        if (it.kind == BATCH_UNPACK) {
            uint16_t* Wm = (uint16_t*)it.dst;
            if (it.M == 4) unpack_group<4>(vals, idx, it.in, it.N, Wm, it.wpr, local);
            else if (it.M == 8) unpack_group<8>(vals, idx, it.in, it.N, Wm, it.wpr, local);
            else unpack_group<16>(vals, idx, it.in, it.N, Wm, it.wpr, local);
        } else {
            uint16_t* a_img = (uint16_t*)it.dst;
            uint16_t* meta16 = (uint16_t*)it.dst2;
            // aux = K blocks of the metadata layout, aux2 = K steps per block, aux3 = layout of the image
            if (it.M == 4) to_sp24_segment<4>(vals, idx, it.out, it.in, it.N, it.wpr, a_img, meta16, it.aux, it.aux2, it.aux3, local);
            else if (it.M == 8) to_sp24_segment<8>(vals, idx, it.out, it.in, it.N, it.wpr, a_img, meta16, it.aux, it.aux2, it.aux3, local);
            else to_sp24_segment<16>(vals, idx, it.out, it.in, it.N, it.wpr, a_img, meta16, it.aux, it.aux2, it.aux3, local);
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
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    long long blocks = (total + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (blocks > (long long)dev.sm_count * 8) blocks = (long long)dev.sm_count * 8;   // one wave of resident blocks
    const unsigned grid = (unsigned)blocks;
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

elsa_status launch_compress_levels(const uint16_t* W, int out, int in, int M, const LevelTable& t, cudaStream_t stream)
{
    const int segs_per_row = (in / M + 31) / 32;
    const long long total = (long long)out * segs_per_row;
    const unsigned grid = (unsigned)((total + kWarpsPerBlock - 1) / kWarpsPerBlock);
    const dim3 block(kWarpsPerBlock * 32);
    ProfileScope scope(ELSA_KERNEL_COMPRESS, stream);
    if (M == 4) launch_pdl(nm_compress_levels_kernel<4>, dim3(grid), block, 0, stream, 1, W, out, in, t, segs_per_row);
    else if (M == 8) launch_pdl(nm_compress_levels_kernel<8>, dim3(grid), block, 0, stream, 1, W, out, in, t, segs_per_row);
    else launch_pdl(nm_compress_levels_kernel<16>, dim3(grid), block, 0, stream, 1, W, out, in, t, segs_per_row);
    return launched("nm_compress (levels)");
}

elsa_status launch_mask(const uint16_t* W, int out, int in, int N, int M, uint16_t* Wm, cudaStream_t stream)
{
    const long long groups = (long long)out * (in / M);
    const unsigned grid = (unsigned)((groups + 255) / 256);
    ProfileScope scope(ELSA_KERNEL_WEIGHT_IMAGES, stream);
    if (M == 4) launch_pdl(nm_mask_kernel<4>, dim3(grid), dim3(256), 0, stream, 1, W, groups, N, Wm);
    else if (M == 8) launch_pdl(nm_mask_kernel<8>, dim3(grid), dim3(256), 0, stream, 1, W, groups, N, Wm);
    else launch_pdl(nm_mask_kernel<16>, dim3(grid), dim3(256), 0, stream, 1, W, groups, N, Wm);
    return launched("nm_mask");
}

// ---- batched launchers

void batch_add_compress(BatchTable* t, const uint16_t* W, int out, int in, int N, int M, uint16_t* vals, uint32_t* idx)
{
    BatchItem& it = t->item[t->n++];
    const int segs_per_row = (in / M + 31) / 32;
    it.src = W; it.src2 = nullptr; it.dst = vals; it.dst2 = idx;
    it.out = out; it.in = in; it.N = N; it.M = M;
    it.wpr = (int)index_words_per_row(in, N, M);
    it.aux = segs_per_row; it.aux2 = 0; it.aux3 = 0; it.kind = BATCH_COMPRESS;
    it.first_unit = t->total_units;
    t->total_units += (long long)out * segs_per_row;
}

void batch_add_unpack(BatchTable* t, const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                      uint16_t* Wm)
{
    BatchItem& it = t->item[t->n++];
    it.src = vals; it.src2 = idx; it.dst = Wm; it.dst2 = nullptr;
    it.out = out; it.in = in; it.N = N; it.M = M;
    it.wpr = (int)index_words_per_row(in, N, M);
    it.aux = 0; it.aux2 = 0; it.aux3 = 0; it.kind = BATCH_UNPACK;
    it.first_unit = t->total_units;
    t->total_units += (long long)out * (in / M);
}

void batch_add_to_sp24(BatchTable* t, const uint16_t* vals, const uint32_t* idx, int out, int in, int N, int M,
                       int block_k, int layout, uint16_t* a_img, uint8_t* meta)
{
    BatchItem& it = t->item[t->n++];
    const int tiles_f = (out + 127) / 128;
    const int k_blocks = (in + block_k - 1) / block_k;
    const int steps = block_k / 32;
    it.src = vals; it.src2 = idx; it.dst = a_img; it.dst2 = meta;
    it.out = out; it.in = in; it.N = N; it.M = M;
    it.wpr = (int)index_words_per_row(in, N, M);
    it.aux = k_blocks; it.aux2 = steps; it.aux3 = layout; it.kind = BATCH_TO_SP24;
    it.first_unit = t->total_units;
    t->total_units += (long long)tiles_f * 128 * k_blocks * steps * 2;
}

elsa_status launch_compress_batch(const BatchTable& t, cudaStream_t stream)
{
    if (t.n == 0) return ELSA_OK;
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    long long grid = (t.total_units + kWarpsPerBlock - 1) / kWarpsPerBlock;
    const long long waves = (long long)dev.sm_count * 4 * 4;   // a few waves of resident blocks (four per SM)
    if (grid > waves) grid = waves;
    ProfileScope scope(ELSA_KERNEL_COMPRESS, stream);
    launch_pdl(nm_compress_batch_kernel, dim3((unsigned)grid), dim3(kWarpsPerBlock * 32), 0, stream, 1, t);
    return launched("nm_compress (batched)");
}

elsa_status launch_image_batch(const BatchTable& t, cudaStream_t stream)
{
    if (t.n == 0) return ELSA_OK;
    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    long long grid = (t.total_units + 255) / 256;
    const long long waves = (long long)dev.sm_count * 8 * 4;
    if (grid > waves) grid = waves;
    ProfileScope scope(ELSA_KERNEL_WEIGHT_IMAGES, stream);
    launch_pdl(nm_image_batch_kernel, dim3((unsigned)grid), dim3(256), 0, stream, 1, t);
    return launched("weight images (batched)");
}

}  // namespace elsa
