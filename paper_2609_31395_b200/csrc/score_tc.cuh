// Tensor-core path of actkv_score (tcgen05 + TMEM + TMA).  Placeholder until the kernels land:
// reports "not supported" so every shape takes the FMA path.
#pragma once

#include "score_fma.cuh"

namespace actkv {

inline bool score_tc_supported(const actkv_pool_t*, int, int) { return false; }

inline int score_tc_launch_lse(ScoreArgs&, const actkv_pool_t*, int, int, cudaStream_t) { return ACTKV_E_INVALID; }
inline int score_tc_launch_score(ScoreArgs&, const actkv_pool_t*, int, int, cudaStream_t) { return ACTKV_E_INVALID; }

}  // namespace actkv
