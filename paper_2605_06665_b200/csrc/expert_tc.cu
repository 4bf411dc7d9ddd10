// placeholder: tensor-core grouped GEMMs land here; bring-up routes to the CUDA-core path.
#include "common.cuh"
namespace unipool {
int tc_module_init(unipool_ctx*) { return UNIPOOL_OK; }
void tc_module_destroy(unipool_ctx*) {}
int expert_fwd_tc(unipool_ctx* c, const ExpertFwdArgs& a, cudaStream_t s) { return expert_fwd_simt(c, a, s); }
int expert_bwd_tc(unipool_ctx* c, const ExpertBwdArgs& a, cudaStream_t s) { return expert_bwd_simt(c, a, s); }
int pool_wgrad_tc(unipool_ctx* c, const PoolWgradArgs& a, cudaStream_t s) { return pool_wgrad_simt(c, a, s); }
}
