// placeholder until the tcgen05 kernel lands
#include "common.cuh"
namespace ada {
bool gram_tc_available() { return false; }
cudaError_t launch_gram_tc(ada_ctx*, const GramProblem&, cudaStream_t) { return cudaErrorNotSupported; }
}
