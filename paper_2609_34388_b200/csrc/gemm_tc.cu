// placeholder until the tcgen05 kernel lands
#include "kernels.h"
namespace recg {
bool launch_gemm_tc(const GemmArgs&, void*, int*, cudaStream_t) { return false; }
void* tc_state_create(int) { return nullptr; }
void tc_state_destroy(void*) {}
}  // namespace recg
