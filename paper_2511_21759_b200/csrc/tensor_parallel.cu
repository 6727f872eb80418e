// Tensor parallelism keeps no kernels of its own on the forward path: the O / down / LM-head projections store
// their results into every rank's buffers and the last CTA of the launch raises this rank's flags
// (tp_arrive_and_signal, called from the GEMM epilogue), and the kernels that consume the exchanged data (RMSNorm,
// the merge of the confidence statistics) begin with a bounded wait on the flags of all ranks (tp_wait_flags).
// Plain loads and stores to peer memory only.  This file holds the test entry that runs the consumers' wait alone.
#include "odb_internal.cuh"

namespace odb {

namespace {

__global__ void __launch_bounds__(32) tp_wait_kernel(TpWait tw) {
    pdl_launch_dependents();
    pdl_wait();
    tp_wait_flags(tw);
}

}  // namespace

cudaError_t launch_tp_wait(const TpWait& tw, cudaStream_t st) {
    if (tw.world < 2 || tw.world > kTpMaxWorld || !tw.region || !tw.status || tw.kind < 0 || tw.kind >= kTpKinds)
        return cudaErrorInvalidValue;
    return launch_kernel(tp_wait_kernel, dim3(1), dim3(32), 0, st, tw);
}

}  // namespace odb
