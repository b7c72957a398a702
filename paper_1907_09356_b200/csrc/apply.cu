// The update half of a CHOCO step (Algorithm 1: public copies, gossip, gradient step; Algorithm 2 for the
// momentum variant): every worker reads its neighbours' messages back and forms
//     x^_i += q_i ;  s_i += sum_j w_ij q_j  (CSR column order, from +0) ;
//     x_i  = (x_i - eta g_i) + gamma (s_i - x^_i).
// This file only picks the kernel: sparse Q goes to the bulk-copy kernel, the rest to the
// dense update kernels.
#include "select.cuh"

namespace choco {

// ---------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------

bool apply_can_emit(const Dev& dv, const StepArgs& a)
{
    if (dv.kind == CHOCO_Q_TOPK) return true;
    if (dv.kind == CHOCO_Q_RANDK) return false;
    return update_dense_can_emit(dv);
}

cudaError_t launch_apply(const Dev& dv, const StepArgs& a, bool emit, cudaStream_t st)
{
    const bool sparse = dv.kind == CHOCO_Q_TOPK || dv.kind == CHOCO_Q_RANDK;
    const cudaError_t e = sparse ? launch_update_bulk(dv, a, emit, st) : launch_update_dense(dv, a, emit, st);
    *a.launches += 1;
    return e != cudaSuccess ? e : cudaGetLastError();
}

} // namespace choco
