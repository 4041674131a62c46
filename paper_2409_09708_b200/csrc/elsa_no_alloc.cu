// elsa_nm_linear_static: the N:M linear for callers that cannot allocate device memory.
//
// Some users of this library run where allocation is off limits: inside a runtime plugin's
// enqueue hook, under a framework that has already claimed the whole device for its own pool, or
// in a loop that must not take the device-wide stall an allocation brings.  They can pass their
// inputs and outputs but have no scratch buffer to give.  For them the weight image that the
// tensor-core kernel reads is rebuilt in the fixed array below, which is part of the library's
// device image: every GPU that loads the library carries it until the process ends.
//
// The array's name means two different things.  In device code it is the array.  In host code it
// is only a handle: handing it to a kernel as a pointer would make the kernel touch host-side
// memory (a fault, or silent garbage on systems where the GPU can reach host memory).  The host
// therefore asks the runtime for the array's device address, once per device, and passes that.
//
// The array is shared by all calls and never cleared.  That is safe because the expand kernel
// writes every element of the [out][in] image (zeros included) before the GEMM reads it; stale
// bytes beyond the image are never read.  Calls that can run concurrently on the GPU would
// overwrite each other's image: they must be ordered on a stream.

#include <mutex>

#include "elsa_internal.h"

namespace elsa {
namespace {

static __device__ __align__(256) unsigned char g_static_scratch[ELSA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// Device address of the scratch array on the current device, looked up on first use.
elsa_status static_scratch(int device, void** out)
{
    if (device < 0 || device >= kMaxDevices)
        return fail(ELSA_ERR_CUDA, "device ordinal %d is outside the %d devices this entry point tracks", device,
                    kMaxDevices);
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[device]) {
        void* ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess || !ptr) {
            cudaGetLastError();
            return fail(ELSA_ERR_CUDA, "cudaGetSymbolAddress for the static scratch array failed on device %d: %s",
                        device, cudaGetErrorString(e));
        }
        g_scratch_addr[device] = ptr;
    }
    *out = g_scratch_addr[device];
    return ELSA_OK;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

}  // namespace
}  // namespace elsa

using namespace elsa;

extern "C" elsa_status elsa_nm_linear_static(const void* X, int rows, const void* vals, const uint32_t* idx,
                                             const void* bias, int out, int in, int N, int M, elsa_dtype dtype,
                                             void* Y, uint32_t* dev_status, void* stream_)
{
    if (!X || !vals || !Y) return fail(ELSA_ERR_NULL, "X, vals and Y must not be NULL");
    if (dtype != ELSA_F16 && dtype != ELSA_BF16)
        return fail(ELSA_ERR_DTYPE, "dtype %d is neither ELSA_F16 nor ELSA_BF16", (int)dtype);
    if (rows <= 0 || out <= 0 || in <= 0)
        return fail(ELSA_ERR_SHAPE, "non-positive dimension (rows=%d, out=%d, in=%d)", rows, out, in);
    if (index_bits(M) < 0 || N < 1 || N > M)
        return fail(ELSA_ERR_NM, "unsupported level %d:%d (M in {4, 8, 16}, 1 <= N <= M)", N, M);
    if (in % M != 0) return fail(ELSA_ERR_SHAPE, "in=%d is not a multiple of M=%d", in, M);
    if (in % 8 != 0 || out % 8 != 0)
        return fail(ELSA_ERR_ALIGN, "in=%d and out=%d must be multiples of 8 (16-byte row pitch)", in, out);
    if (N != M && !idx) return fail(ELSA_ERR_NULL, "idx must not be NULL when N < M");
    if (!aligned16(X) || !aligned16(vals) || !aligned16(Y) || (idx && !aligned16(idx)) || (bias && !aligned16(bias)))
        return fail(ELSA_ERR_ALIGN, "X, vals, idx, bias and Y must be 16-byte aligned");
    const size_t image_bytes = (size_t)out * (size_t)in * 2;
    if (N != M && image_bytes > (size_t)ELSA_STATIC_SCRATCH_BYTES)
        return fail(ELSA_ERR_WORKSPACE,
                    "weight image of %zu bytes (out=%d x in=%d x 2) exceeds the built-in scratch of %u bytes; "
                    "use elsa_nm_linear with a caller-provided workspace",
                    image_bytes, out, in, (unsigned)ELSA_STATIC_SCRATCH_BYTES);

    DeviceInfo dev;
    elsa_status st = device_info(&dev);
    if (st != ELSA_OK) return st;
    cudaStream_t stream = (cudaStream_t)stream_;

    const uint16_t* Wd = (const uint16_t*)vals;  // the dense level is multiplied as stored
    if (N != M) {
        void* scratch = nullptr;
        if ((st = static_scratch(dev.device, &scratch)) != ELSA_OK) return st;
        // rebuilds all out*in elements of the image: nothing left by an earlier call survives in it
        if ((st = launch_unpack((const uint16_t*)vals, idx, out, in, N, M, (uint16_t*)scratch, stream)) != ELSA_OK)
            return st;
        Wd = (const uint16_t*)scratch;
    }
    return launch_linear_tc_dense((const uint16_t*)X, rows, Wd, (const uint16_t*)bias, out, in, dtype, (uint16_t*)Y,
                                  dev_status, stream);
}
