// Flags between the ranks of a tensor-parallel group.  The data itself (fp32 partial tiles of the O and down
// projections, confidence statistics of the LM head) is stored into every rank's receive buffers by the
// projection's epilogue (gemm_tcgen05.cu, PeerOut); these two one-warp kernels order it: a rank raises its flag on
// every rank once its stores are visible system-wide, and waits (bounded) for the flags of all ranks before the
// kernel that adds the partials up.  Plain loads and stores to peer memory only.
#include "odb_internal.cuh"

namespace odb {

namespace {

__device__ __forceinline__ void st_release_sys(unsigned int* p, unsigned int v) {
    asm volatile("st.release.sys.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ unsigned int ld_acquire_sys(const unsigned int* p) {
    unsigned int v;
    asm volatile("ld.acquire.sys.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}

__global__ void __launch_bounds__(32) tp_signal_kernel(TpPeers p, int kind, unsigned int seq) {
    pdl_launch_dependents();
    pdl_wait();   // the projection whose epilogue stored to the peers has completed
    __threadfence_system();
    if (static_cast<int>(threadIdx.x) < p.world)
        st_release_sys(p.flags[threadIdx.x] + kind * kTpMaxWorld + p.rank, seq);
}

__global__ void __launch_bounds__(32) tp_wait_kernel(TpPeers p, int kind, unsigned int seq, long long limit_cycles, int* status) {
    pdl_launch_dependents();
    pdl_wait();
    if (static_cast<int>(threadIdx.x) < p.world) {
        const unsigned int* f = p.flags[p.rank] + kind * kTpMaxWorld + threadIdx.x;
        const long long t0 = clock64();
        // sequence numbers only grow; the signed difference keeps the comparison valid across a wrap
        while (static_cast<int>(ld_acquire_sys(f) - seq) < 0) {
            if (clock64() - t0 > limit_cycles) {
                atomicExch(status, ODB_ERR_TIMEOUT);
                break;
            }
            __nanosleep(64);
        }
    }
    __threadfence_system();
}

}  // namespace

cudaError_t launch_tp_signal(const TpPeers& p, int kind, unsigned int seq, cudaStream_t st) {
    if (p.world < 2 || p.world > kTpMaxWorld || kind < 0 || kind >= kTpKinds) return cudaErrorInvalidValue;
    return launch_kernel(tp_signal_kernel, dim3(1), dim3(32), 0, st, p, kind, seq);
}

cudaError_t launch_tp_wait(const TpPeers& p, int kind, unsigned int seq, long long limit_cycles, int* status, cudaStream_t st) {
    if (p.world < 2 || p.world > kTpMaxWorld || kind < 0 || kind >= kTpKinds) return cudaErrorInvalidValue;
    return launch_kernel(tp_wait_kernel, dim3(1), dim3(32), 0, st, p, kind, seq, limit_cycles, status);
}

}  // namespace odb
