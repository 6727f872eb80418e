// odb_gemm_static_scratch: the weight-streaming GEMM for callers that cannot allocate device
// memory.  The split-K partial sums, which every other entry point keeps in a caller-provided
// buffer, live here in a fixed array that is part of the library image on the device.
#include <mutex>

#include "odb_internal.cuh"

using namespace odb;

namespace {

constexpr size_t kScratchBytes = ODB_STATIC_SCRATCH_BYTES;   // partial sums
constexpr size_t kStatusBytes = 256;                          // device status word behind them

// Resident on every GPU that loads the library, from load until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes + kStatusBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device

// In host code the name `g_static_scratch` is only a handle for the runtime, not an address the
// GPU can use: the device address has to be asked for, once per device, with that device current.
cudaError_t scratch_address(unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_ptr[dev] = static_cast<unsigned char*>(p);
    }
    *out = g_scratch_ptr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" int32_t odb_gemm_static_scratch(const void* x, const void* w_packed, float* out, int32_t M, int32_t N,
                                           int32_t K, int32_t k_splits, void* stream) {
    if (!x || !w_packed || !out) return ODB_ERR_ARG;
    if (M < 1 || N < 1 || K < 8 || K % 8) return ODB_ERR_SHAPE;
    int splits = k_splits > 0 ? k_splits : gemm_pick_splits(M, N, K);
    const int nkb = (K + 63) / 64;
    if (splits > nkb) splits = nkb;
    while (splits > 1 && ((nkb + splits - 1) / splits) * (splits - 1) >= nkb) --splits;
    // the fixed array bounds the problem: splits * M * N partial sums of 4 bytes
    if (static_cast<size_t>(splits) * M * N * sizeof(float) > kScratchBytes) return ODB_ERR_WORKSPACE;

    unsigned char* scratch = nullptr;
    cudaError_t e = scratch_address(&scratch);
    if (e != cudaSuccess) return ODB_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int* status = reinterpret_cast<int*>(scratch + kScratchBytes);
    // The array keeps whatever the previous call left.  The partial sums need no clearing (every
    // element that is read back is written first by this call's splits); the status word does.
    if (cudaMemsetAsync(status, 0, sizeof(int), st) != cudaSuccess) return ODB_ERR_CUDA;

    GemmArgs ga;
    if (make_weight_tmap(&ga.tmap_w, w_packed, N, K) != cudaSuccess) return ODB_ERR_CUDA;
    ga.x = x;
    ga.partial = reinterpret_cast<float*>(scratch);
    ga.act_out = nullptr;
    ga.M = M; ga.N = N; ga.K = K;
    ga.splits = splits;
    ga.status = status;
    if (launch_gemm(ga, st) != cudaSuccess) return ODB_ERR_CUDA;
    if (launch_reduce_partials(ga.partial, splits, static_cast<size_t>(M) * N, out, static_cast<size_t>(M) * N, st) !=
        cudaSuccess)
        return ODB_ERR_CUDA;
    int host_status = 0;
    if (cudaMemcpyAsync(&host_status, status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess) return ODB_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return ODB_ERR_CUDA;
    return host_status;
}
