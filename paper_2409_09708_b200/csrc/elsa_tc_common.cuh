// Pieces shared by the tensor-core linear kernels: inline-PTX wrappers for mbarriers, TMA, tcgen05 and
// tensor memory, the shared-memory matrix descriptor, and the host-side tensor-map encoder.
// Included by each kernel's translation unit; everything here has internal linkage.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include "elsa_internal.h"

namespace elsa {
namespace {

constexpr unsigned long long kWaitTimeoutNs = 2000000000ull;  // 2 s per wait

// ------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}

__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// Bounded wait.  Returns false if this wait, or any other wait of the CTA, has given up: after `limit_ns`
// the waiter sets the CTA's abort flag and records ELSA_ERR_TIMEOUT | site << 8 in `dev_status`.
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                                uint32_t* dev_status, uint32_t site, unsigned long long limit_ns)
{
    uint32_t spins = 0;
    unsigned long long t0 = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 0xFFu) == 0) {
            if (*abort_flag) return false;
            const unsigned long long now = global_timer_ns();
            if (t0 == 0) {
                t0 = now;
            } else if (now - t0 > limit_ns) {
                *abort_flag = 1;
                if (dev_status) atomicCAS(dev_status, 0u, (uint32_t)ELSA_ERR_TIMEOUT | (site << 8));
                return false;
            }
        }
    }
    return true;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                          uint32_t* dev_status, uint32_t site)
{
    return mbar_wait_limit(bar, parity, abort_flag, dev_status, site, kWaitTimeoutNs);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0,
                                            int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src, int c0, int c1)
{
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(map)),
                 "r"(src), "r"(c0), "r"(c1)
                 : "memory");
}

__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }

template <int kPending>
__device__ __forceinline__ void bulk_wait_group_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kPending) : "memory");
}

__device__ __forceinline__ void bulk_wait_group_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t holder, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// D[tmem] (+)= A[smem] * B[smem]^T, both operands K-major.
__device__ __forceinline__ void umma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                         uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// The mbarrier receives one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
                 : "memory");
}

// Lane i of the warp receives 32 consecutive fp32 columns of TMEM lane (lane base + i).
__device__ __forceinline__ void tmem_ld_32x32b_x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]),
          "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]),
          "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]),
          "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile stored as rows of 128 bytes with the 128-byte
// swizzle (what TMA writes): 8-row groups are 1024 bytes apart; start address in 16-byte units.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw128(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);        // start address
    d |= (uint64_t)1 << 16;                        // leading byte offset: unused with swizzle
    d |= (uint64_t)(1024 >> 4) << 32;              // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                        // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                        // layout: 128-byte swizzle
    return d;
}

// Shared-memory matrix descriptor of an MN-major tile: rows of 128 bytes (64 16-bit values along M or N) per
// reduction index, written by TMA with the 128-byte swizzle.  8 reduction rows form a 1024-byte group (stride
// offset); blocks of 64 values along M / N are `block_bytes` apart (leading offset).
__device__ __forceinline__ uint64_t smem_desc_mn_major_sw128(uint32_t addr, uint32_t block_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((block_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

template <bool kBf16>
__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    if constexpr (kBf16) {
        __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    } else {
        __half2 v = __floats2half2_rn(lo, hi);
        return *reinterpret_cast<uint32_t*>(&v);
    }
}

// Two 16-bit values packed in a word (low half first) as floats.
template <bool kBf16>
__device__ __forceinline__ float2 raw2_to_float2(uint32_t w)
{
    if constexpr (kBf16) return make_float2(__uint_as_float(w << 16), __uint_as_float(w & 0xFFFF0000u));
    else return __half22float2(*reinterpret_cast<const __half2*>(&w));
}

// GELU in its exact form, v * Phi(v) = 0.5 v (1 + erf(v / sqrt 2)) (the activation of the ViT MLP), in fp32.
// With a = |v|: gelu(v) = max(v, 0) - 0.5 a erfc(a / sqrt 2), and erfc(a / sqrt 2) = 2^Q(a) with Q a polynomial of
// degree 6 fitted to log2 erfc on [0, 5.9375] (beyond it erfc < 3e-9; fit_gelu.py beside the package's build script
// reproduces the coefficients and the error: 3e-7 absolute in fp32 over all v).  Ten instructions and one
// special-function-unit operation per value; the library erff cost the epilogue warps about 40 instructions and
// tripled the time of an fc1 layer on the sparse kernels, a rational form with a reciprocal still doubled it.
__device__ __forceinline__ float gelu_exact(float v)
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

// Epilogue activation of a layer: 0 none, 1 GELU.
__device__ __forceinline__ float apply_act(float v, int act) { return act == 1 ? gelu_exact(v) : v; }

template <bool kBf16>
__device__ __forceinline__ float bias_to_float(uint16_t u)
{
    if constexpr (kBf16) return __bfloat162float(__ushort_as_bfloat16(u));
    else return __half2float(__ushort_as_half(u));
}


// ------------------------------------------------------------------ CTA-pair (cluster of two) forms

__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}

// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one()
{
    uint32_t e;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xFFFFFFFF;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(e));
    return e != 0;
}

// Address, in the cluster's shared window, of this CTA's shared address `addr` inside CTA `rank`.
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }

// Arrive on an mbarrier that may live in the other CTA of the pair.  The arrival hands back tensor
// memory whose reads have already completed (tcgen05.wait::ld, tcgen05.fence::before_thread_sync), so
// it orders nothing in ordinary memory: the default CTA-scope release is enough, and a cluster-scope
// release here cost the epilogue ~0.6 us per tile waiting for its own stores to drain.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}

// TMA load into this CTA's shared memory whose completion bytes are credited to an mbarrier that may
// live in the other CTA of the pair.
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
        : "memory");
}

__device__ __forceinline__ void tmem_alloc_pair(uint32_t holder, uint32_t cols)
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(holder), "r"(cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

// One MMA over the pair: M = 256 (128 rows of A from each CTA), B rows split between the two CTAs,
// each CTA's tensor memory receives its 128 rows of D.  Issued by the leader CTA only.
__device__ __forceinline__ void umma_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// One arrival on the mbarrier at this shared offset in every CTA of `cta_mask`, once all MMAs issued
// so far by this thread have completed.
__device__ __forceinline__ void umma_commit_pair(uint32_t bar, uint16_t cta_mask)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                 "h"(cta_mask)
                 : "memory");
}

// ------------------------------------------------------------------ 2:4-sparse MMA forms

// D[tmem] (+)= A[smem, 2:4-compressed along K] * B[smem]^T.  `tmem_e` is the tensor-memory column
// holding the metadata of this K step; the column's parity goes into the instruction descriptor's
// sparsity selector and the even column address into the operand.
__device__ __forceinline__ void umma_sp_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t tmem_e,
                                            uint32_t idesc, uint32_t accumulate)
{
    const uint32_t idesc_sel = idesc | (tmem_e & 1u);
    const uint32_t e_addr = tmem_e & ~1u;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "tcgen05.mma.sp.cta_group::1.kind::f16 [%0], %1, %2, [%3], %4, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(e_addr), "r"(idesc_sel), "r"(accumulate)
        : "memory");
}

// Copies 128 rows x 16 bytes from shared memory (descriptor) into 4 consecutive columns of the 128
// lanes of tensor memory.  Ordered with the MMAs issued by the same thread.
__device__ __forceinline__ void tmem_cp_128x128b(uint32_t taddr, uint64_t s_desc)
{
    asm volatile("tcgen05.cp.cta_group::1.128x128b [%0], %1;" ::"r"(taddr), "l"(s_desc) : "memory");
}

// Plain (untiled) bulk copy global -> shared, completion counted on an mbarrier.  Addresses and size
// are multiples of 16 bytes.
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

// K-major tile stored as rows of 64 bytes with the 64-byte swizzle: 8-row groups are 512 bytes apart.
__device__ __forceinline__ uint64_t smem_desc_k_major_sw64(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(512 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)4 << 61;   // layout: 64-byte swizzle
    return d;
}

// Unswizzled K-major block of 16-byte rows: 8 rows are 128 contiguous bytes, 8-row groups follow
// each other.
__device__ __forceinline__ uint64_t smem_desc_rows16_no_swizzle(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)(128 >> 4) << 16;   // leading byte offset (one 16-byte column only: unused)
    d |= (uint64_t)(128 >> 4) << 32;   // stride between 8-row groups
    d |= (uint64_t)1 << 46;
    return d;
}

// CTA-pair forms of the two above: M = 256 (128 compressed rows of A and their metadata from each
// CTA), B rows split between the CTAs; the copy runs in both CTAs, each from its own shared memory
// into its own tensor memory.  Issued by the leader CTA.
__device__ __forceinline__ void umma_sp_f16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t tmem_e,
                                                 uint32_t idesc, uint32_t accumulate)
{
    const uint32_t idesc_sel = idesc | (tmem_e & 1u);
    const uint32_t e_addr = tmem_e & ~1u;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(e_addr), "r"(idesc_sel), "r"(accumulate)
        : "memory");
}

__device__ __forceinline__ void tmem_cp_128x128b_pair(uint32_t taddr, uint64_t s_desc)
{
    asm volatile("tcgen05.cp.cta_group::2.128x128b [%0], %1;" ::"r"(taddr), "l"(s_desc) : "memory");
}

// Plain bulk copy whose completion bytes go to an mbarrier that may live in the other CTA of the pair.
__device__ __forceinline__ void bulk_load_1d_pair(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar_cluster_addr)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar_cluster_addr)
                 : "memory");
}

// ------------------------------------------------------------------ tensor-memory operand forms (weight held in TMEM)

// A from tensor memory: lane = weight row, 8 columns per K step of 32 (16 kept values of 16 bits).
// Called by the whole (converged) warp; `issue` is non-zero in the one lane that issues.  The predicate
// lives inside the asm block so that the compiler cannot turn it into a branch around the instruction.
__device__ __forceinline__ void umma_sp_f16_pair_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t tmem_e,
                                                    uint32_t idesc, uint32_t accumulate, uint32_t issue)
{
    const uint32_t idesc_sel = idesc | (tmem_e & 1u);
    const uint32_t e_addr = tmem_e & ~1u;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "setp.ne.b32 q, %6, 0;\n"
        "@q tcgen05.mma.sp.cta_group::2.kind::f16 [%0], [%1], %2, [%3], %4, p;\n"
        "}\n" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(e_addr), "r"(idesc_sel), "r"(accumulate), "r"(issue)
        : "memory");
}

// Lane i of the warp receives 16 consecutive fp32 columns of TMEM lane (lane base + i).
__device__ __forceinline__ void tmem_ld_32x32b_x16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// Four 8 x 8 matrices of 16-bit values, transposed on the way to shared memory: the two halves of
// register i of lane t go to column t / 4 of rows 2 * (t % 4) and 2 * (t % 4) + 1 of matrix i, whose
// eight 16-byte rows are at the addresses given by lanes 8 * i .. 8 * i + 7.
__device__ __forceinline__ void stmatrix_x4_trans(uint32_t addr, uint32_t r0, uint32_t r1, uint32_t r2, uint32_t r3)
{
    asm volatile("stmatrix.sync.aligned.m8n8.x4.trans.shared.b16 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(r0), "r"(r1),
                 "r"(r2), "r"(r3)
                 : "memory");
}

// Lane i of the warp writes 16 / 4 consecutive columns of TMEM lane (lane base + i).
__device__ __forceinline__ void tmem_st_32x32b_x16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
        "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
        "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__device__ __forceinline__ void tmem_st_32x32b_x4(uint32_t taddr, const uint32_t (&r)[4])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1, %2, %3, %4};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
                 "r"(r[2]), "r"(r[3])
                 : "memory");
}

// 3-D TMA load into this CTA's shared memory, completion bytes credited to an mbarrier that may live in
// the other CTA of the pair.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster_addr, int c0,
                                                 int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Arrival that publishes this CTA's tensor-memory writes to the MMA issuer of the leader CTA.
__device__ __forceinline__ void mbar_arrive_cluster_release(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}


// ------------------------------------------------------------------ forms predicated on the issuing lane
//
// The tensor-core instructions below are executed by a whole converged warp with `issue` non-zero in one
// elected lane.  The predicate sits on the instruction inside the asm block: written as `if (elected) mma`
// the compiler branches around every instruction, which measured ~80 cycles per MMA in the issuing warp
// against ~36 for the predicated form.

__device__ __forceinline__ void umma_f16_if(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
        : "memory");
}

__device__ __forceinline__ void umma_commit_if(uint32_t bar, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred q;\n"
        "setp.ne.b32 q, %1, 0;\n"
        "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n"
        "}\n" ::"r"(bar),
        "r"(issue)
        : "memory");
}

__device__ __forceinline__ void umma_f16_pair_if(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
        : "memory");
}

// The same for 8-bit integer operands (K = 32 per instruction, int32 accumulators).
__device__ __forceinline__ void umma_i8_pair_if(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                uint32_t accumulate, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "setp.ne.b32 q, %5, 0;\n"
        "@q tcgen05.mma.cta_group::2.kind::i8 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
        : "memory");
}

__device__ __forceinline__ void umma_commit_pair_if(uint32_t bar, uint16_t cta_mask, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred q;\n"
        "setp.ne.b32 q, %2, 0;\n"
        "@q tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n"
        "}\n" ::"r"(bar),
        "h"(cta_mask), "r"(issue)
        : "memory");
}

__device__ __forceinline__ void umma_sp_f16_pair_if(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t tmem_e,
                                                    uint32_t idesc, uint32_t accumulate, uint32_t issue)
{
    const uint32_t idesc_sel = idesc | (tmem_e & 1u);
    const uint32_t e_addr = tmem_e & ~1u;
    asm volatile(
        "{\n"
        ".reg .pred p, q;\n"
        "setp.ne.b32 p, %5, 0;\n"
        "setp.ne.b32 q, %6, 0;\n"
        "@q tcgen05.mma.sp.cta_group::2.kind::f16 [%0], %1, %2, [%3], %4, p;\n"
        "}\n" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(e_addr), "r"(idesc_sel), "r"(accumulate), "r"(issue)
        : "memory");
}

__device__ __forceinline__ void tmem_cp_128x128b_pair_if(uint32_t taddr, uint64_t s_desc, uint32_t issue)
{
    asm volatile(
        "{\n"
        ".reg .pred q;\n"
        "setp.ne.b32 q, %2, 0;\n"
        "@q tcgen05.cp.cta_group::2.128x128b [%0], %1;\n"
        "}\n" ::"r"(taddr),
        "l"(s_desc), "r"(issue)
        : "memory");
}

// ------------------------------------------------------------------ host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn lookup_encode_tiled()
{
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
        return reinterpret_cast<EncodeTiledFn>(ptr);
    return nullptr;
}

// Looked up once; a function-local static is initialised exactly once even when several host threads make
// their first tensor-core call together.
EncodeTiledFn encode_tiled_fn()
{
    static const EncodeTiledFn fn = lookup_encode_tiled();
    return fn;
}

// 2-D row-major 16-bit tensor [dim1][dim0], box [box1][box0].
elsa_status make_map_2d(CUtensorMap* map, const void* base, uint64_t dim0, uint64_t dim1, uint32_t box0,
                        uint32_t box1, CUtensorMapSwizzle swizzle, const char* what)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(ELSA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {dim0 * 2};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t elem[2] = {1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, elem,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ELSA_ERR_CUDA, "tensor map for %s rejected (CUresult %d)", what, (int)rc);
    return ELSA_OK;
}

// 2-D row-major 8-bit tensor [dim1][dim0], box [box1][box0].
elsa_status make_map_2d_u8(CUtensorMap* map, const void* base, uint64_t dim0, uint64_t dim1, uint32_t box0,
                           uint32_t box1, CUtensorMapSwizzle swizzle, const char* what)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(ELSA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[2] = {dim0, dim1};
    cuuint64_t strides[1] = {dim0};
    cuuint32_t box[2] = {box0, box1};
    cuuint32_t elem[2] = {1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, elem,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ELSA_ERR_CUDA, "tensor map for %s rejected (CUresult %d)", what, (int)rc);
    return ELSA_OK;
}

// Row-major 16-bit matrix [rows][in] seen as [in / 64][rows][64]: one box of (64, box_rows, box_quarters) is a
// K stage of 64 * box_quarters as that many 128-byte-swizzled quarters of box_rows rows each.
elsa_status make_map_x_quarters(CUtensorMap* map, const void* base, uint64_t in, uint64_t rows, uint32_t box_rows,
                                uint32_t box_quarters)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return fail(ELSA_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    cuuint64_t dims[3] = {64, rows, in / 64};
    cuuint64_t strides[2] = {in * 2, 128};
    cuuint32_t box[3] = {64, box_rows, box_quarters};
    cuuint32_t elem[3] = {1, 1, 1};
    CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT16, 3, const_cast<void*>(base), dims, strides, box, elem,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(ELSA_ERR_CUDA, "tensor map for X rejected (CUresult %d)", (int)rc);
    return ELSA_OK;
}



}  // namespace
}  // namespace elsa
