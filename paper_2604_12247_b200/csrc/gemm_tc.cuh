// Interface of the TMA + tcgen05 weight-streaming kernels (bf16 models).
#pragma once
#include <cuda_runtime.h>

#include <map>
#include <vector>

#include "sb_internal.cuh"

namespace sb {

constexpr int kMaxSplit = kMaxSplitK;   // most split-K partials a GEMM may leave for its consumer

struct TcPlan;                 // tensor maps + work decomposition of one GEMM call shape
struct TcPlanCache {
    std::map<std::vector<uint64_t>, TcPlan*> plans;
    void clear();
    ~TcPlanCache() { clear(); }
};

bool tc_available();
// one CTA waits (bounded by budget_cycles) on a barrier nothing completes; status receives code 9, waited_flag 2
void launch_wait_selftest(cudaStream_t st, unsigned int* status, unsigned long long budget_cycles, unsigned int* waited_flag);
// pipeline depth (2..12 stages of 18 KB) and persistent CTAs per SM (1..2) of the launches that follow
bool tc_set_tuning(int stages, int ctas_per_sm);
// a GEMM that announces a later pair-mode GEMM (GemmArgs::next_*) prefetches every n-th k block of that GEMM's
// weights into L2 while it waits for its own predecessor; 0 = never
bool tc_set_l2_prefetch(int every);
// cost the host's work decomposition charges for each additional k split, per mille of the streaming time
bool tc_set_split_penalty(int per_mille);
// wide passes (GemmArgs::nb > 1): true (default) = clusters of two CTAs sharing one activation tile (cta_group::2),
// false = one CTA per work item
void tc_set_wide_cta_pairs(bool on);
// the work decomposition for `units` CTAs (modes 0, 1: 8-row kernel, its gate/up form) or clusters (modes 2, 3: CTA-pair
// kernel, its gate/up form): rows per CTA (gate/up: columns per item), k splits, work items.  Host arithmetic only.
bool tc_plan_query(int mode, const int* n_rows, int n_mats, int K, int units, int* R, int* S, int* n_items);
// returns the number of split-K partials written to a.out, or -1 if no TMA descriptor could be made
int launch_gemm_tc(cudaStream_t st, const GemmArgs& a, TcPlanCache* cache, unsigned int* status);
bool launch_head_tc(cudaStream_t st, const HeadArgs& a, TcPlanCache* cache, unsigned int* status);

}  // namespace sb
