#include "gemm_tc.cuh"
namespace sb {
struct TcPlan {};
void TcPlanCache::clear() { for (auto& kv : plans) delete kv.second; plans.clear(); }
bool tc_available() { return false; }
int launch_gemm_tc(cudaStream_t, const GemmArgs&, TcPlanCache*, unsigned int*) { return 0; }
void launch_head_tc(cudaStream_t, const HeadArgs&, TcPlanCache*, unsigned int*) {}
}
