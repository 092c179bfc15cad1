// Cluster row-statistics kernel (placeholder until the optimised variant lands): reports "not
// applicable" so that every shape takes the baseline kernel.
#pragma once

#include "common.cuh"

namespace psd {

inline bool cluster_kernel_applicable(const StageParams&, int) { return false; }
inline int launch_rowstats_cluster(const StageParams&, int, cudaStream_t) { return -2; }
inline int cluster_occupancy(int, int, int* cs, int* n) {
  if (cs) *cs = 0;
  if (n) *n = 0;
  return 0;
}

}  // namespace psd
