// fathom_klt_basis: eigenbasis and eigenvalues of the 128 x 128 key covariance of every KV head (Sec. 3.5 "Basis rule";
// Appendix B5: mean, eigenbasis and eigenvalues of a layer's keys from the session's own prefill cache), so that a rotated
// store can be built with library calls alone: fathom_calibrate -> fathom_klt_basis -> fathom_rotate_keys / _query.
//
// Two-sided cyclic Jacobi, one CTA per KV head, everything in shared memory: the symmetric matrix A in fp64 (128 KB), the
// accumulated rotations V in fp32 (64 KB).  A sweep is 127 steps of 64 disjoint pairs (p, q) in round-robin order (player
// 127 stays, the others move round a ring), so every pair meets once per sweep and the 64 rotations of a step commute:
//   rotation  64 threads: t = sgn(theta) / (|theta| + sqrt(theta^2 + 1)), theta = (a_qq - a_pp) / (2 a_pq), c, s;
//   columns   A <- A J and V <- V J  (all 1024 threads, 128 rows x 64 pairs);
//   rows      A <- J^T A             (128 columns x 64 pairs).
// Sweeps stop when the off-diagonal mass has fallen below 1e-24 of the diagonal's (at most 16 sweeps; a covariance of
// keys takes 7 or 8).  The order of operations is fixed, so the result is bit-reproducible.  Eigenvalues come out
// in descending order (ties: lower original index first) and every direction is signed so that its largest component is
// positive; the rotated store does not depend on either choice.  Eigenvalues are clamped at zero.
#include "fathom_common.cuh"

namespace {

constexpr int EIG_THREADS = 1024;
constexpr int N = FATHOM_D;                                   // 128
constexpr int LDA = N + 1;                                    // padded rows of A: column walks hit different banks
constexpr int MAX_SWEEPS = 16;

struct EigSmem {
  double A[N * LDA];
  float V[N * LDA];
  double c[N / 2], s[N / 2];
  int p[N / 2], q[N / 2];
  double red[EIG_THREADS / 32][2];
  double off2, diag2;
  int rank[N];
};

__global__ void __launch_bounds__(EIG_THREADS, 1)
klt_eig_kernel(const float* __restrict__ cov, float* __restrict__ basis, float* __restrict__ eigenvalues) {
  extern __shared__ __align__(16) unsigned char raw[];
  EigSmem& M = *reinterpret_cast<EigSmem*>(raw);
  const int kv = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* C = cov + (size_t)kv * N * N;

  for (int e = tid; e < N * N; e += EIG_THREADS) {
    const int i = e >> 7, j = e & (N - 1);
    M.A[i * LDA + j] = 0.5 * ((double)C[i * N + j] + (double)C[j * N + i]);    // the symmetric part, exactly
    M.V[i * LDA + j] = i == j ? 1.0f : 0.0f;
  }
  __syncthreads();

  for (int sweep = 0; sweep < MAX_SWEEPS; ++sweep) {
    // ---- how far from diagonal?  (fixed-order reduction: per thread, per warp, then thread 0)
    {
      double off = 0.0, dg = 0.0;
      for (int e = tid; e < N * N; e += EIG_THREADS) {
        const int i = e >> 7, j = e & (N - 1);
        const double a = M.A[i * LDA + j];
        if (i == j) dg += a * a; else off += a * a;
      }
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        off += __shfl_xor_sync(0xffffffffu, off, o);
        dg += __shfl_xor_sync(0xffffffffu, dg, o);
      }
      if (lane == 0) { M.red[warp][0] = off; M.red[warp][1] = dg; }
      __syncthreads();
      if (tid == 0) {
        double o2 = 0.0, d2 = 0.0;
        for (int w = 0; w < EIG_THREADS / 32; ++w) { o2 += M.red[w][0]; d2 += M.red[w][1]; }
        M.off2 = o2; M.diag2 = d2;
      }
      __syncthreads();
      if (M.off2 <= 1e-24 * M.diag2) break;                    // uniform over the CTA
    }
    for (int step = 0; step < N - 1; ++step) {
      // ---- the 64 pairs of this step and their rotations
      if (tid < N / 2) {
        int p, q;
        if (tid == 0) { p = step; q = N - 1; }
        else { p = (step + tid) % (N - 1); q = (step - tid + (N - 1)) % (N - 1); }
        if (p > q) { const int t = p; p = q; q = t; }
        const double apq = M.A[p * LDA + q], app = M.A[p * LDA + p], aqq = M.A[q * LDA + q];
        double c = 1.0, s = 0.0;
        if (fabs(apq) > 1e-300) {
          const double theta = (aqq - app) / (2.0 * apq);
          const double t = (theta >= 0.0 ? 1.0 : -1.0) / (fabs(theta) + sqrt(theta * theta + 1.0));
          c = 1.0 / sqrt(t * t + 1.0);
          s = t * c;
        }
        M.p[tid] = p; M.q[tid] = q; M.c[tid] = c; M.s[tid] = s;
      }
      __syncthreads();
      // ---- columns: A <- A J, V <- V J
      {
        const int k = tid & 63;
        const int p = M.p[k], q = M.q[k];
        const double c = M.c[k], s = M.s[k];
        const float cf = (float)c, sf = (float)s;
#pragma unroll
        for (int m = 0; m < N / 16; ++m) {
          const int i = (tid >> 6) + 16 * m;
          const double ap = M.A[i * LDA + p], aq = M.A[i * LDA + q];
          M.A[i * LDA + p] = c * ap - s * aq;
          M.A[i * LDA + q] = s * ap + c * aq;
          const float vp = M.V[i * LDA + p], vq = M.V[i * LDA + q];
          M.V[i * LDA + p] = __fsub_rn(__fmul_rn(cf, vp), __fmul_rn(sf, vq));
          M.V[i * LDA + q] = __fadd_rn(__fmul_rn(sf, vp), __fmul_rn(cf, vq));
        }
      }
      __syncthreads();
      // ---- rows: A <- J^T A
      {
        const int j = tid & (N - 1);
#pragma unroll
        for (int m = 0; m < N / 16; ++m) {
          const int k = (tid >> 7) + 8 * m;
          const int p = M.p[k], q = M.q[k];
          const double c = M.c[k], s = M.s[k];
          const double ap = M.A[p * LDA + j], aq = M.A[q * LDA + j];
          M.A[p * LDA + j] = c * ap - s * aq;
          M.A[q * LDA + j] = s * ap + c * aq;
        }
      }
      __syncthreads();
    }
  }

  // ---- eigenvalues in descending order (ties: lower index first); direction j goes to column rank[j], signed so that its
  //      largest component is positive
  if (tid < N) {
    const double mine = M.A[tid * LDA + tid];
    int r = 0;
    for (int i = 0; i < N; ++i) {
      const double other = M.A[i * LDA + i];
      r += (other > mine || (other == mine && i < tid)) ? 1 : 0;
    }
    M.rank[tid] = r;
    eigenvalues[(size_t)kv * N + r] = (float)fmax(mine, 0.0);   // a variance: rounding may leave -1e-20 on a rank-deficient input
    float big = 0.0f;
    for (int i = 0; i < N; ++i) {
      const float v = M.V[i * LDA + tid];
      if (fabsf(v) > fabsf(big)) big = v;
    }
    reinterpret_cast<float*>(M.red)[tid] = big < 0.0f ? -1.0f : 1.0f;   // (the reduction buffer is free now)
  }
  __syncthreads();
  for (int e = tid; e < N * N; e += EIG_THREADS) {
    const int i = e >> 7, j = e & (N - 1);
    basis[(size_t)kv * N * N + i * N + M.rank[j]] = M.V[i * LDA + j] * reinterpret_cast<const float*>(M.red)[j];
  }
}

}  // namespace

extern "C" int fathom_klt_basis(fathom_ctx* ctx, const fathom_layout* L, const float* cov, float* basis, float* eigenvalues,
                                void* stream) {
  if (!ctx || !cov || !basis || !eigenvalues) return FATHOM_ERR_INVALID_ARG;
  const int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (!fathom_aligned16(cov) || !fathom_aligned16(basis)) return FATHOM_ERR_ALIGNMENT;
  static bool configured[64] = {};
  int dev = 0;
  FATHOM_CUDA_TRY(ctx, cudaGetDevice(&dev));
  if (dev >= 0 && dev < 64 && !configured[dev]) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(klt_eig_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(EigSmem)));
    configured[dev] = true;
  }
  klt_eig_kernel<<<L->n_kv_heads, EIG_THREADS, sizeof(EigSmem), static_cast<cudaStream_t>(stream)>>>(cov, basis, eigenvalues);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
