// tasc_gemm_bf16_static: the tensor-core product of tasc_gemm_bf16 for callers that must not allocate.
//
// Some hosts of this library cannot obtain device memory at the moment they need a product: code
// running inside a fixed-memory serving process whose pool was handed out at start-up, a plugin
// whose host forbids cudaMalloc after initialisation, or a caller that simply has no allocator at
// hand to size the split-K workspace tasc_gemm_bf16 asks for.  For them the split-K partial sums
// live in one file-scope device array of fixed size that every GPU loading the library keeps until
// the process exits.  The caller still supplies inputs and output.
//
// The array is shared by every call: it keeps whatever the previous call left, two calls that run
// concurrently on one GPU (different streams, or threads) overwrite each other's partial sums, and
// products whose partial sums do not fit are refused rather than spilled anywhere else.
#include "kernels.h"

#include <mutex>

namespace tasc {
namespace {

constexpr size_t STATIC_SCRATCH_BYTES = 8u << 20;      // 8 MiB per GPU
constexpr size_t STATUS_BYTES = 256;                   // first bytes: the device status word

static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[MAX_DEVICES];            // device address of the array on each GPU, once looked up

// In host code `g_static_scratch` names a host-side shadow of the symbol, not memory a kernel can use;
// the address kernels need comes from the runtime, per device, with that device current.
tasc_status scratch_for_current_device(unsigned char** out) {
    int dev = -1;
    TASC_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= MAX_DEVICES) return TASC_EINVAL;
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        TASC_CUDA_TRY(cudaGetSymbolAddress(&p, g_static_scratch));
        if (!p || (reinterpret_cast<uintptr_t>(p) % 256)) return TASC_ECUDA;
        tasc_status st = gemm_set_attributes();
        if (st != TASC_OK) return st;
        g_scratch_addr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_addr[dev];
    return TASC_OK;
}

}  // namespace
}  // namespace tasc

using namespace tasc;

extern "C" tasc_status tasc_gemm_bf16_static(const void* x, const void* wt, float* y, int32_t M, int32_t N, int32_t K,
                                             int32_t* device_status, tasc_stream stream) {
    if (!x || !wt || !y || M < 1 || N < 1 || K < 8 || K % 8) return TASC_EINVAL;
    const size_t room = STATIC_SCRATCH_BYTES - STATUS_BYTES;
    // Fewer k-splits than tasc_gemm_bf16 would take are fine (only the summation order changes);
    // a product whose single-split output does not fit has no place to go.
    const GemmPlan p = plan_gemm(M, N, K, room, false);
    if (gemm_partial_bytes(p, M, N) > room) return TASC_ECAPACITY;
    unsigned char* scratch = nullptr;
    tasc_status st = scratch_for_current_device(&scratch);
    if (st != TASC_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    CUtensorMap tmW, tmX;
    if ((st = encode_tmap_bf16(&tmW, wt, N, K, 128)) != TASC_OK) return st;
    if ((st = encode_tmap_bf16(&tmX, x, M, K, p.BN)) != TASC_OK) return st;
    // The status word starts at zero for every call; the partial sums need no clearing because the
    // kernel writes every element the reduction reads.
    int* status = device_status ? device_status : reinterpret_cast<int*>(scratch);
    TASC_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int), s));
    float* partials = reinterpret_cast<float*>(scratch + STATUS_BYTES);
    if ((st = launch_gemm_bf16(&tmW, &tmX, partials, M, N, K, p, status, s)) != TASC_OK) return st;
    launch_sum_partials(partials, p.splits, y, (size_t)M * N, s);
    TASC_CUDA_TRY(cudaGetLastError());
    return TASC_OK;
}
