// fathom_alloc_depth: per-plan read depths (Sec. 3.3, Eq. 3 and Eq. 4; fixed-channel rule of Sec. 2).
//
// Eq. 4 at the smallest water line that fits the budget grants exactly the min(B, 4d) candidate planes
// (channel j, plane m = 1..4) with the largest priority g_j 4^-m, so a candidate is granted when fewer than
// B others rank before it (ties: lower channel, then lower plane).  Four CTAs of 512 threads serve a plan:
// every CTA computes all 128 importances (thread = channel; fp64 with explicit round-to-nearest intrinsics,
// no fused multiply-add, so the ranking is identical on every machine; no logarithm is evaluated) and ranks
// the 128 candidates of its own 32 channels against all 512, four threads per candidate (each counts over a
// quarter of the others: the kernel is a latency chain, and the counting loop is its longest link).
// Non-negative doubles order like their bit patterns, so the comparisons run on 64-bit integers.
#include "fathom_common.cuh"

namespace {

constexpr int NCAND = FATHOM_D * FATHOM_NPLANES;   // 512
constexpr int CTAS_PER_PLAN = 4;
constexpr int AD_CAND = NCAND / CTAS_PER_PLAN;     // 128 candidates ranked per CTA
constexpr int AD_SPLIT = 4;                        // threads per candidate
constexpr int AD_THREADS = AD_CAND * AD_SPLIT;     // 512

__global__ void __launch_bounds__(AD_THREADS)
alloc_depth_kernel(const float* __restrict__ q, const float* __restrict__ var, int mode, int budget,
                   int heads_per_plan, int G, uint8_t* __restrict__ depth) {
  __shared__ alignas(16) unsigned long long pri[NCAND];       // bit patterns of the (non-negative) priorities
  __shared__ int partial[AD_SPLIT][AD_CAND];
  FATHOM_PDL_WAIT();
  FATHOM_PDL_RELEASE();                                       // the scan that follows may become resident now
  const int plan = blockIdx.x / CTAS_PER_PLAN, part = blockIdx.x % CTAS_PER_PLAN;
  const int tid = threadIdx.x;
  const int h0 = plan * heads_per_plan;
  const int kv = h0 / G;
  uint8_t* out = depth + (size_t)plan * FATHOM_D;

  if (mode == FATHOM_DEPTH_UNIFORM) {
    if (part == 0 && tid < FATHOM_D) out[tid] = (uint8_t)min(max(budget, 0), FATHOM_NPLANES);
    return;
  }

  if (tid < FATHOM_D) {                                       // thread = channel: its four priorities
    const int j = tid;
    double acc = 0.0;
    if (mode == FATHOM_DEPTH_WATERFILL) {
      for (int h = h0; h < h0 + heads_per_plan; ++h) {
        const double x = (double)q[(size_t)h * FATHOM_D + j];
        acc = __dadd_rn(acc, __dmul_rn(x, x));                // Eq. 3, heads in ascending order
      }
      const double g = __dmul_rn(acc, (double)var[(size_t)kv * FATHOM_D + j]);
      pri[4 * j + 0] = (unsigned long long)__double_as_longlong(fabs(__dmul_rn(g, 0.25)));        // g_j 4^-m
      pri[4 * j + 1] = (unsigned long long)__double_as_longlong(fabs(__dmul_rn(g, 0.0625)));
      pri[4 * j + 2] = (unsigned long long)__double_as_longlong(fabs(__dmul_rn(g, 0.015625)));
      pri[4 * j + 3] = (unsigned long long)__double_as_longlong(fabs(__dmul_rn(g, 0.00390625)));
    } else {                                                  // fixed top-r channels by sum_h |q_j|
      for (int h = h0; h < h0 + heads_per_plan; ++h)
        acc = __dadd_rn(acc, fabs((double)q[(size_t)h * FATHOM_D + j]));
      const unsigned long long key = (unsigned long long)__double_as_longlong(acc);
      pri[4 * j + 0] = key; pri[4 * j + 1] = key; pri[4 * j + 2] = key; pri[4 * j + 3] = key;
    }
  }
  __syncthreads();

  const int cand = tid & (AD_CAND - 1), quarter = tid / AD_CAND;
  const int id = part * AD_CAND + cand;                       // my candidate: channel id / 4, plane id % 4 + 1
  const unsigned long long key = pri[id];
  int rank = 0;
  const int o0 = quarter * (NCAND / AD_SPLIT), o1 = o0 + NCAND / AD_SPLIT;
  if (mode == FATHOM_DEPTH_WATERFILL) {
#pragma unroll 8
    for (int o = o0; o < o1; o += 2) {
      const ulonglong2 p = *reinterpret_cast<const ulonglong2*>(&pri[o]);
      rank += (p.x > key) || (p.x == key && o < id);
      rank += (p.y > key) || (p.y == key && o + 1 < id);
    }
  } else {                                                    // rank channels only (one key per channel)
#pragma unroll 8
    for (int o = o0; o < o1; o += 4) {
      const unsigned long long p = pri[o];
      rank += (p > key) || (p == key && o < (id & ~3));
    }
  }
  partial[quarter][cand] = rank;
  __syncthreads();
  if (quarter == 0) {                                         // the first four warps: one thread per candidate
    rank = partial[0][cand] + partial[1][cand] + partial[2][cand] + partial[3][cand];
    const bool granted = rank < budget;                       // fixed mode: all four planes of a chosen channel
    const unsigned ball = __ballot_sync(0xffffffffu, granted);
    if ((id & 3) == 0) out[id >> 2] = (uint8_t)__popc((ball >> (tid & 31)) & 0xFu);
  }
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
  alloc_depth_kernel<<<plans * CTAS_PER_PLAN, AD_THREADS, 0, static_cast<cudaStream_t>(stream)>>>(q, var, mode, budget, heads_per_plan, G, depth);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
