// fathom_alloc_depth: per-plan read depths (Sec. 3.3, Eq. 3 and Eq. 4; fixed-channel rule of Sec. 2).
//
// One CTA of 4 * 128 threads per plan; thread (j, m) owns candidate plane m = 1..4 of channel j.
// Eq. 4 at the smallest water line that fits the budget grants exactly the min(B, 4d) candidate
// planes with the largest priority g_j 4^-m, so each thread ranks its own candidate against the
// other 511 (ties: lower channel, then lower plane) and is granted when its rank is below B.  All
// arithmetic is fp64 with explicit round-to-nearest intrinsics (no fused multiply-add), so the
// ranking is identical on every machine; no logarithm is evaluated.
#include "fathom_common.cuh"

namespace {

constexpr int NCAND = FATHOM_D * FATHOM_NPLANES;   // 512

__global__ void __launch_bounds__(NCAND)
alloc_depth_kernel(const float* __restrict__ q, const float* __restrict__ var, int mode, int budget,
                   int heads_per_plan, int G, uint8_t* __restrict__ depth) {
  __shared__ double pri[NCAND];
  const int plan = blockIdx.x;
  const int tid = threadIdx.x;
  const int j = tid >> 2;             // channel
  const int m = (tid & 3) + 1;        // candidate plane 1..4
  const int h0 = plan * heads_per_plan;
  const int kv = h0 / G;
  uint8_t* out = depth + (size_t)plan * FATHOM_D;

  if (mode == FATHOM_DEPTH_UNIFORM) {
    if (m == 1) out[j] = (uint8_t)min(max(budget, 0), FATHOM_NPLANES);
    return;
  }

  double key;
  if (mode == FATHOM_DEPTH_WATERFILL) {
    double acc = 0.0;
    for (int h = h0; h < h0 + heads_per_plan; ++h) {
      const double x = (double)q[(size_t)h * FATHOM_D + j];
      acc = __dadd_rn(acc, __dmul_rn(x, x));                  // Eq. 3, heads in ascending order
    }
    const double g = __dmul_rn(acc, (double)var[(size_t)kv * FATHOM_D + j]);
    const double scale = (m == 1) ? 0.25 : (m == 2) ? 0.0625 : (m == 3) ? 0.015625 : 0.00390625;
    key = __dmul_rn(g, scale);                                // g_j 4^-m
  } else {                                                    // fixed top-r channels by sum_h |q_j|
    double acc = 0.0;
    for (int h = h0; h < h0 + heads_per_plan; ++h)
      acc = __dadd_rn(acc, fabs((double)q[(size_t)h * FATHOM_D + j]));
    key = acc;
  }
  pri[tid] = key;
  __syncthreads();

  bool granted;
  if (mode == FATHOM_DEPTH_WATERFILL) {
    int rank = 0;
    for (int o = 0; o < NCAND; ++o) {
      const double p = pri[o];
      rank += (p > key) || (p == key && o < tid);
    }
    granted = rank < budget;
  } else {
    int rank = 0;                                             // rank channels only (candidate m = 1 of each)
    for (int o = 0; o < NCAND; o += 4) {
      const double p = pri[o];
      rank += (p > key) || (p == key && o < (tid & ~3));
    }
    granted = rank < budget;                                  // all four planes of a chosen channel
  }
  const unsigned ball = __ballot_sync(0xffffffffu, granted);
  if (m == 1) out[j] = (uint8_t)__popc((ball >> (threadIdx.x & 31)) & 0xFu);
}

}  // namespace

extern "C" int fathom_alloc_depth(fathom_ctx* ctx, const fathom_layout* L, const float* q, const float* var,
                                  int mode, int budget, int heads_per_plan, uint8_t* depth, void* stream) {
  if (!ctx || !q || !depth) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (mode != FATHOM_DEPTH_WATERFILL && mode != FATHOM_DEPTH_FIXED_TOP_R && mode != FATHOM_DEPTH_UNIFORM)
    return FATHOM_ERR_UNSUPPORTED;
  if (mode == FATHOM_DEPTH_WATERFILL && !var) return FATHOM_ERR_INVALID_ARG;
  if (budget < 0) return FATHOM_ERR_INVALID_ARG;
  if (mode == FATHOM_DEPTH_UNIFORM && budget > FATHOM_NPLANES) return FATHOM_ERR_INVALID_ARG;
  const int G = L->n_q_heads / L->n_kv_heads;
  if (heads_per_plan < 1 || G % heads_per_plan != 0) return FATHOM_ERR_INVALID_ARG;
  const int plans = L->n_q_heads / heads_per_plan;
  alloc_depth_kernel<<<plans, NCAND, 0, static_cast<cudaStream_t>(stream)>>>(q, var, mode, budget, heads_per_plan, G, depth);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
