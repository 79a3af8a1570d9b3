// The method's schedule, host side: which scale steps run densely, which run under the fidelity-refinement
// approximation and which are skipped (Sec. 4.1), the rank of every block group at a late scale (App. A.1,
// the table of mean rank ratios for alpha = 0.96) and the rank that a ratio stands for (Sec. 3.2,
// Eq. "low_rank_percent": a ratio is a fraction of n = min(M, d)).  No device code.
#include <math.h>

#include "../../include/fvar.h"

namespace {

constexpr int kInfinityScales[13] = {1, 2, 4, 6, 8, 12, 16, 20, 24, 32, 40, 48, 64};
constexpr int kInfinityLate[3] = {40, 48, 64};
constexpr double kInfinityAlpha[3] = {0.96, 0.0, 0.0};        // Sec. 4.1: one threshold per late scale; 0 skips the step

// App. A.1: rows = block chunk 0..7, columns = scale 40, 48, 64 (alpha = 0.96)
constexpr double kRankRatio096[8][3] = {
    {0.016, 0.013, 0.008}, {0.136, 0.117, 0.054}, {0.210, 0.189, 0.083}, {0.250, 0.222, 0.066},
    {0.256, 0.234, 0.056}, {0.198, 0.183, 0.029}, {0.157, 0.134, 0.038}, {0.191, 0.163, 0.055},
};

int late_column(int scale_side) {
  for (int i = 0; i < 3; ++i)
    if (kInfinityLate[i] == scale_side) return i;
  return -1;
}

int clamp_rank(double v, int M) {
  const int r = static_cast<int>(floor(v + 0.5));
  return r < 1 ? 1 : (r > M ? M : r);
}

}  // namespace

extern "C" {

int fvar_rank_from_keep_ratio(int M, float keep_ratio) {
  if (M <= 0) return 0;
  const int r = static_cast<int>(floorf(keep_ratio * M + 0.5f));
  return r < 1 ? 1 : (r > M ? M : r);
}

int fvar_rank_from_table_ratio(int M, int width, double ratio) {
  if (M <= 0 || width <= 0) return 0;
  return clamp_rank(ratio * (M < width ? M : width), M);
}

fvar_status fvar_infinity_rank_ratio(int chunk, int scale_side, double *ratio_host) {
  const int col = late_column(scale_side);
  if (chunk < 0 || chunk >= 8 || col < 0 || !ratio_host) return FVAR_EINVAL;
  *ratio_host = kRankRatio096[chunk][col];
  return FVAR_OK;
}

fvar_status fvar_infinity_group_ranks(int scale_side, int width, int n_groups, int *ranks_host) {
  const int col = late_column(scale_side);
  if (col < 0 || width <= 0 || n_groups <= 0 || !ranks_host) return FVAR_EINVAL;
  const int M = scale_side * scale_side;
  for (int g = 0; g < n_groups; ++g) {
    int chunk = static_cast<int>((g + 0.5) * 8 / n_groups);      // the chunk at the nearest relative depth
    chunk = chunk > 7 ? 7 : chunk;
    ranks_host[g] = fvar_rank_from_table_ratio(M, width, kRankRatio096[chunk][col]);
  }
  return FVAR_OK;
}

fvar_status fvar_infinity_schedule(int paper_schedule, int capacity, int *sides_host, int *modes_host, int *count_host) {
  if (!count_host || capacity < 0) return FVAR_EINVAL;
  *count_host = 13;
  for (int k = 0; k < 13 && k < capacity; ++k) {
    const int col = late_column(kInfinityScales[k]);
    if (sides_host) sides_host[k] = kInfinityScales[k];
    if (modes_host)
      modes_host[k] = col < 0 ? FVAR_DENSE : ((!paper_schedule || kInfinityAlpha[col] > 0.0) ? FVAR_LOWRANK_RTR : FVAR_SKIP);
  }
  return FVAR_OK;
}

}  // extern "C"
