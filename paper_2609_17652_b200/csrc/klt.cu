// KLT-rotated store (Sec. 3.5 "Basis rule") and session calibration (Appendix B5).
//
//   fathom_channel_variance  per-channel mean and variance of a session's keys (the raw store's Var(k_j));
//   fathom_calibrate      mean and covariance of a session's own keys, one covariance per KV head;
//   fathom_rotate_keys    K' = (K - mu) V, the keys whose planes the rotated variant stores;
//   fathom_rotate_query   q' = q V, from which g_j = sum_h (q'_hj)^2 lambda_j is formed by fathom_alloc_depth
//                         (eigenvalues passed as `var`).
//
// This file holds the statistics kernels, the entry points and the plain-fp32 variants of rotation and covariance
// (FATHOM_ROTATE_PATH=simt, FATHOM_CALIBRATE_PATH=simt); the default paths are the tcgen05 kernels of klt_tc.cu, which
// split both operands into tf32 head and tail so that the rotated keys, which feed a quantiser, keep fp32 accuracy.
// The fp32 variants are the same register-tiled product  C[i][j] += P[t][i] * Q[t][j]  over a shared-memory panel:
// 256 threads, each an 8 x 8 block of the 128 x 128 result (columns split 4 + 4 so that the 16-byte panel loads of
// neighbouring lanes are contiguous), plain FMAs in a fixed order.
#include "fathom_common.cuh"

#include <cstdlib>
#include <cstring>

namespace {

constexpr int KT_THREADS = 256;
constexpr int PANEL = FATHOM_D + 4;                          // floats per panel row (16-byte aligned, staggers banks)
constexpr int COV_ROWS = 8192;                               // rows per CTA of the covariance pass
constexpr int MEAN_ROWS = 1024;                              // rows per CTA of the mean pass

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

// acc[i][j] += sum_t P[t][8 ty + i] * Q[t][cols(tx, j)],  cols = 4 tx + j (j < 4), 64 + 4 tx + (j - 4) (j >= 4)
__device__ __forceinline__ void panel_product(const float* __restrict__ P, const float* __restrict__ Q, int T, int ty, int tx,
                                              float (&acc)[8][8]) {
#pragma unroll 4
  for (int t = 0; t < T; ++t) {
    const float4 a0 = *reinterpret_cast<const float4*>(P + t * PANEL + 8 * ty);
    const float4 a1 = *reinterpret_cast<const float4*>(P + t * PANEL + 8 * ty + 4);
    const float4 b0 = *reinterpret_cast<const float4*>(Q + t * PANEL + 4 * tx);
    const float4 b1 = *reinterpret_cast<const float4*>(Q + t * PANEL + 64 + 4 * tx);
    const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
    const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
  }
}

// ---- K' = (K - mu) V : one CTA per 128 tokens of one KV head -------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(KT_THREADS)
rotate_keys_kernel(const T* __restrict__ K, const float* __restrict__ mean, const float* __restrict__ basis,
                   float* __restrict__ K_rot, long long n) {
  extern __shared__ __align__(16) float sm[];
  float* As = sm;                                             // [c][row]: the token tile, transposed, mean removed
  float* Bs = sm + FATHOM_D * PANEL;                          // [c][j]  : the basis
  const int kv = blockIdx.y, tid = threadIdx.x;
  const long long r0 = (long long)blockIdx.x * FATHOM_D;
  const T* Kh = K + ((size_t)kv * (size_t)n + (size_t)r0) * FATHOM_D;
  const float* V = basis + (size_t)kv * FATHOM_D * FATHOM_D;
  const float* mu = mean + (size_t)kv * FATHOM_D;
  for (int e = tid; e < FATHOM_D * (FATHOM_D / 4); e += KT_THREADS) {        // basis rows, 16 bytes a piece
    const int c = e / (FATHOM_D / 4), j4 = e % (FATHOM_D / 4);
    *reinterpret_cast<float4*>(Bs + c * PANEL + 4 * j4) = __ldg(reinterpret_cast<const float4*>(V + c * FATHOM_D) + j4);
  }
  // token tile: lane = row (so the transposed stores of a warp are conflict-free), 4 channels per step
  for (int e = tid; e < FATHOM_D * (FATHOM_D / 4); e += KT_THREADS) {
    const int row = e % FATHOM_D, c4 = e / FATHOM_D;
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    if (r0 + row < n) {
#pragma unroll
      for (int x = 0; x < 4; ++x) v[x] = to_f32(Kh[(size_t)row * FATHOM_D + 4 * c4 + x]) - mu[4 * c4 + x];
    }
#pragma unroll
    for (int x = 0; x < 4; ++x) As[(4 * c4 + x) * PANEL + row] = v[x];
  }
  __syncthreads();
  const int ty = tid >> 4, tx = tid & 15;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;
  panel_product(As, Bs, FATHOM_D, ty, tx, acc);
  float* out = K_rot + ((size_t)kv * (size_t)n + (size_t)r0) * FATHOM_D;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = 8 * ty + i;
    if (r0 + row < n) {
      *reinterpret_cast<float4*>(out + (size_t)row * FATHOM_D + 4 * tx) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
      *reinterpret_cast<float4*>(out + (size_t)row * FATHOM_D + 64 + 4 * tx) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
    }
  }
}

// ---- q' = q V ---------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(FATHOM_D)
rotate_query_kernel(const float* __restrict__ q, const float* __restrict__ basis, float* __restrict__ q_rot, int G) {
  __shared__ float s_q[FATHOM_D];
  const int h = blockIdx.x, j = threadIdx.x;
  const float* V = basis + (size_t)(h / G) * FATHOM_D * FATHOM_D;
  s_q[j] = q[(size_t)h * FATHOM_D + j];
  __syncthreads();
  float acc = 0.0f;
#pragma unroll 8
  for (int c = 0; c < FATHOM_D; ++c) acc = fmaf(s_q[c], __ldg(V + c * FATHOM_D + j), acc);
  q_rot[(size_t)h * FATHOM_D + j] = acc;
}

// ---- calibration ------------------------------------------------------------------------------------------------
// (1) the mean from the one-pass statistics kernels below; (2) partial (K - mu)^T (K - mu) of COV_ROWS tokens;
// (3) their fp64 sum in tile order / (n - 1) -> covariance.
template <typename T>
__global__ void __launch_bounds__(KT_THREADS)
cov_partial_kernel(const T* __restrict__ K, long long n, const float* __restrict__ mean, float* __restrict__ partial, int tiles) {
  extern __shared__ __align__(16) float sm[];
  float* Xs = sm;                                             // [row][c], mean removed, 128 rows at a time
  const int kv = blockIdx.y, tid = threadIdx.x;
  const long long t0 = (long long)blockIdx.x * COV_ROWS;
  const long long t1 = min(t0 + COV_ROWS, n);
  const T* Kh = K + (size_t)kv * (size_t)n * FATHOM_D;
  const float* mu = mean + (size_t)kv * FATHOM_D;
  const int ty = tid >> 4, tx = tid & 15;
  float acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.0f;
  for (long long r0 = t0; r0 < t1; r0 += FATHOM_D) {
    __syncthreads();
    for (int e = tid; e < FATHOM_D * (FATHOM_D / 4); e += KT_THREADS) {      // consecutive threads = consecutive channels
      const int row = e / (FATHOM_D / 4), c4 = e % (FATHOM_D / 4);
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      if (r0 + row < t1) {
        const T* src = Kh + (size_t)(r0 + row) * FATHOM_D + 4 * c4;
        v = make_float4(to_f32(src[0]) - mu[4 * c4], to_f32(src[1]) - mu[4 * c4 + 1], to_f32(src[2]) - mu[4 * c4 + 2],
                        to_f32(src[3]) - mu[4 * c4 + 3]);
      }
      *reinterpret_cast<float4*>(Xs + row * PANEL + 4 * c4) = v;
    }
    __syncthreads();
    panel_product(Xs, Xs, FATHOM_D, ty, tx, acc);            // rows past the end are zero and add nothing
  }
  float* out = partial + ((size_t)kv * tiles + blockIdx.x) * FATHOM_D * FATHOM_D;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = 8 * ty + i;
    *reinterpret_cast<float4*>(out + row * FATHOM_D + 4 * tx) = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
    *reinterpret_cast<float4*>(out + row * FATHOM_D + 64 + 4 * tx) = make_float4(acc[i][4], acc[i][5], acc[i][6], acc[i][7]);
  }
}

__global__ void __launch_bounds__(FATHOM_D)
cov_final_kernel(const float* __restrict__ partial, int tiles, long long n, float* __restrict__ cov) {
  const int kv = blockIdx.y, i = blockIdx.x, j = threadIdx.x;
  double s = 0.0;
#pragma unroll 8
  for (int t = 0; t < tiles; ++t) s += (double)partial[(((size_t)kv * tiles + t) * FATHOM_D + i) * FATHOM_D + j];
  cov[((size_t)kv * FATHOM_D + i) * FATHOM_D + j] = (float)(s / (double)(n > 1 ? n - 1 : 1));
}

// ---- per-channel mean and variance (the Var(k_j) of the importance g_j) -----------------------------------------
// One pass over the keys.  A CTA takes MEAN_ROWS tokens of one KV head and, per channel, the sums of (x - s) and
// (x - s)^2 with s the tile's middle key (a shift inside the data keeps the squares free of cancellation); the
// final kernel merges the tiles in fp64 in tile order: mean_t = s + S1/n_t, M2_t = S2 - S1^2/n_t,
// M2 = sum M2_t + sum n_t (mean_t - mean)^2.
__device__ __forceinline__ float4 load4(const float* p) { return __ldg(reinterpret_cast<const float4*>(p)); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  const uint2 u = __ldg(reinterpret_cast<const uint2*>(p));
  return make_float4(__uint_as_float(u.x << 16), __uint_as_float(u.x & 0xffff0000u), __uint_as_float(u.y << 16),
                     __uint_as_float(u.y & 0xffff0000u));
}

template <typename T>
__global__ void __launch_bounds__(KT_THREADS)
var_partial_kernel(const T* __restrict__ K, long long n, float* __restrict__ partial, int tiles) {
  __shared__ float4 s_sum[8][32], s_sq[8][32];
  const int kv = blockIdx.y, tid = threadIdx.x, cq = tid & 31, rl = tid >> 5;   // warp = row lane, lane = 4 channels
  const long long r0 = (long long)blockIdx.x * MEAN_ROWS;
  const long long r1 = min(r0 + MEAN_ROWS, n);
  const T* Kh = K + (size_t)kv * (size_t)n * FATHOM_D + 4 * cq;
  const float4 sh = load4(Kh + (size_t)(r0 + (r1 - r0) / 2) * FATHOM_D);   // the tile's middle key (a prompt's first keys may be far off)
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
#pragma unroll 8
  for (long long r = r0 + rl; r < r1; r += 8) {
    const float4 x = load4(Kh + (size_t)r * FATHOM_D);
    const float dx = x.x - sh.x, dy = x.y - sh.y, dz = x.z - sh.z, dw = x.w - sh.w;
    a.x += dx; a.y += dy; a.z += dz; a.w += dw;
    b.x = fmaf(dx, dx, b.x); b.y = fmaf(dy, dy, b.y); b.z = fmaf(dz, dz, b.z); b.w = fmaf(dw, dw, b.w);
  }
  s_sum[rl][cq] = a;
  s_sq[rl][cq] = b;
  __syncthreads();
  if (rl == 0) {
#pragma unroll
    for (int w = 1; w < 8; ++w) {                                // row lanes in a fixed order
      const float4 u = s_sum[w][cq], v = s_sq[w][cq];
      a.x += u.x; a.y += u.y; a.z += u.z; a.w += u.w;
      b.x += v.x; b.y += v.y; b.z += v.z; b.w += v.w;
    }
    float* out = partial + ((size_t)kv * tiles + blockIdx.x) * 3 * FATHOM_D + 4 * cq;
    *reinterpret_cast<float4*>(out) = sh;
    *reinterpret_cast<float4*>(out + FATHOM_D) = a;
    *reinterpret_cast<float4*>(out + 2 * FATHOM_D) = b;
  }
}

// 1024 threads per KV head: thread (channel, lane) merges tiles lane, lane + 8, ... and the eight lanes are then
// combined in lane order, so the result does not depend on scheduling.
constexpr int VF_LANES = 8;
__global__ void __launch_bounds__(FATHOM_D * VF_LANES)
var_final_kernel(const float* __restrict__ partial, int tiles, long long n, float* __restrict__ mean, float* __restrict__ var) {
  __shared__ double s_acc[VF_LANES][FATHOM_D];
  __shared__ double s_mu[FATHOM_D];
  const int kv = blockIdx.x, c = threadIdx.x & (FATHOM_D - 1), tl = threadIdx.x >> 7;
  const float* P = partial + (size_t)kv * tiles * 3 * FATHOM_D + c;
  double total = 0.0;
#pragma unroll 4
  for (int t = tl; t < tiles; t += VF_LANES) {
    const double nt = (double)min((long long)MEAN_ROWS, n - (long long)t * MEAN_ROWS);
    total += nt * (double)P[(size_t)t * 3 * FATHOM_D] + (double)P[(size_t)t * 3 * FATHOM_D + FATHOM_D];
  }
  s_acc[tl][c] = total;
  __syncthreads();
  if (tl == 0) {
    double sum = 0.0;
#pragma unroll
    for (int w = 0; w < VF_LANES; ++w) sum += s_acc[w][c];
    s_mu[c] = sum / (double)n;
  }
  __syncthreads();
  const double mu = s_mu[c];
  double m2 = 0.0;
#pragma unroll 4
  for (int t = tl; t < tiles; t += VF_LANES) {
    const double nt = (double)min((long long)MEAN_ROWS, n - (long long)t * MEAN_ROWS);
    const double s1 = (double)P[(size_t)t * 3 * FATHOM_D + FATHOM_D], s2 = (double)P[(size_t)t * 3 * FATHOM_D + 2 * FATHOM_D];
    const double dm = (double)P[(size_t)t * 3 * FATHOM_D] + s1 / nt - mu;
    m2 += (s2 - s1 * s1 / nt) + nt * dm * dm;
  }
  __syncthreads();
  s_acc[tl][c] = m2;
  __syncthreads();
  if (tl == 0) {
    double sum = 0.0;
#pragma unroll
    for (int w = 0; w < VF_LANES; ++w) sum += s_acc[w][c];
    mean[(size_t)kv * FATHOM_D + c] = (float)mu;
    var[(size_t)kv * FATHOM_D + c] = (float)(sum > 0.0 ? sum / (double)(n > 1 ? n - 1 : 1) : 0.0);
  }
}

// reduction of the tensor-core partials (fp64, slot order): S = sum_t sums[kv][t], mean = shift + S / n,
// cov = (sum_t (P1 + P2 + P2^T) - S S^T / n) / (n - 1)  with the partials [kv][t][2][d][d] of the shifted keys
__global__ void __launch_bounds__(FATHOM_D)
cov_final_tc_kernel(const float* __restrict__ partial, const float* __restrict__ partial_sum, const float* __restrict__ shift,
                    int slots, long long n, float* __restrict__ mean, float* __restrict__ cov) {
  __shared__ double s_S[FATHOM_D];
  const int kv = blockIdx.y, i = blockIdx.x, j = threadIdx.x;
  {
    double t = 0.0;
    for (int u = 0; u < slots; ++u) t += (double)partial_sum[((size_t)kv * slots + u) * FATHOM_D + j];
    s_S[j] = t;
    if (i == 0) mean[(size_t)kv * FATHOM_D + j] = (float)((double)shift[(size_t)kv * FATHOM_D + j] + t / (double)n);
  }
  __syncthreads();
  const float* P = partial + (size_t)kv * slots * 2 * FATHOM_D * FATHOM_D;
  double s = 0.0;
#pragma unroll 4
  for (int t = 0; t < slots; ++t) {
    const float* p1 = P + (size_t)t * 2 * FATHOM_D * FATHOM_D;
    const float* p2 = p1 + FATHOM_D * FATHOM_D;
    s += (double)p1[i * FATHOM_D + j] + ((double)p2[i * FATHOM_D + j] + (double)p2[j * FATHOM_D + i]);
  }
  s -= s_S[i] * s_S[j] / (double)n;
  cov[((size_t)kv * FATHOM_D + i) * FATHOM_D + j] = (float)(s / (double)(n > 1 ? n - 1 : 1));
}

}  // namespace

static size_t stats_partial_bytes(int Hkv, long long n) {
  return fathom_round_up((size_t)Hkv * (size_t)((n + MEAN_ROWS - 1) / MEAN_ROWS) * 3 * FATHOM_D * 4, 256);
}

// covariance partial slots per head: 8192-token tiles of the plain kernel, or the CTAs of the tensor-core kernel
// (at most one per SM over all heads; 256 bounds the SM count)
static size_t cov_partial_slots(int Hkv, long long n) {
  const size_t ct = (size_t)((n + COV_ROWS - 1) / COV_ROWS);
  const size_t tc = 2 * (size_t)(256 / Hkv > 0 ? 256 / Hkv : 1);   // two matrices per CTA
  return ct > tc ? ct : tc;
}

// per-CTA channel sums of the tensor-core covariance pass: at most 256 CTAs over all heads
static size_t cov_sums_bytes() { return (size_t)256 * FATHOM_D * 4; }

size_t fathom_calib_scratch_bytes(int Hkv, long long n) {
  return stats_partial_bytes(Hkv, n) + fathom_round_up((size_t)Hkv * cov_partial_slots(Hkv, n) * FATHOM_D * FATHOM_D * 4, 256) +
         fathom_round_up((size_t)Hkv * FATHOM_D * 4, 256) + cov_sums_bytes();
}

extern "C" int fathom_channel_variance(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, float* mean, float* var,
                                       void* stream) {
  if (!ctx || !K || !mean || !var) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K)) return FATHOM_ERR_ALIGNMENT;
  const int Hkv = L->n_kv_heads;
  const long long n = L->n;
  if (fathom_calib_scratch_bytes(Hkv, n) > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  const int mt = (int)((n + MEAN_ROWS - 1) / MEAN_ROWS);
  float* part = static_cast<float*>(ctx->scratch);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (k_dtype == FATHOM_F32)
    var_partial_kernel<float><<<dim3(mt, Hkv), KT_THREADS, 0, st>>>(static_cast<const float*>(K), n, part, mt);
  else
    var_partial_kernel<__nv_bfloat16><<<dim3(mt, Hkv), KT_THREADS, 0, st>>>(static_cast<const __nv_bfloat16*>(K), n, part, mt);
  var_final_kernel<<<Hkv, FATHOM_D * VF_LANES, 0, st>>>(part, mt, n, mean, var);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_calibrate(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, float* mean, float* cov,
                                void* stream) {
  if (!ctx || !K || !mean || !cov) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K) || !fathom_aligned16(cov)) return FATHOM_ERR_ALIGNMENT;
  const int Hkv = L->n_kv_heads;
  const long long n = L->n;
  if (fathom_calib_scratch_bytes(Hkv, n) > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  const int mt = (int)((n + MEAN_ROWS - 1) / MEAN_ROWS);
  const size_t cov_bytes = fathom_round_up((size_t)Hkv * cov_partial_slots(Hkv, n) * FATHOM_D * FATHOM_D * 4, 256);
  char* base = static_cast<char*>(ctx->scratch);
  float* part = reinterpret_cast<float*>(base);
  float* pcov = reinterpret_cast<float*>(base + stats_partial_bytes(Hkv, n));
  float* var_tmp = reinterpret_cast<float*>(base + stats_partial_bytes(Hkv, n) + cov_bytes);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const char* path = getenv("FATHOM_CALIBRATE_PATH");
  if (!(path && strcmp(path, "simt") == 0)) {
    // tensor cores, ONE read of the keys: covariance and per-channel sums of the keys centred on a shift
    int slots = fathom_cov_tc_ctas_per_head(Hkv);
    if ((size_t)slots * 2 > cov_partial_slots(Hkv, n)) slots = (int)(cov_partial_slots(Hkv, n) / 2);
    float* psum = reinterpret_cast<float*>(base + stats_partial_bytes(Hkv, n) + cov_bytes + fathom_round_up((size_t)Hkv * FATHOM_D * 4, 256));   // [Hkv][slots][d]
    rc = fathom_launch_cov_tc(ctx, L, K, k_dtype, var_tmp, pcov, psum, slots, st);
    if (rc != FATHOM_OK) return rc;
    cov_final_tc_kernel<<<dim3(FATHOM_D, Hkv), FATHOM_D, 0, st>>>(pcov, psum, var_tmp, slots, n, mean, cov);
    FATHOM_CUDA_TRY(ctx, cudaGetLastError());
    return FATHOM_OK;
  }
  // plain fp32 kernels: (1) mean
  if (k_dtype == FATHOM_F32)
    var_partial_kernel<float><<<dim3(mt, Hkv), KT_THREADS, 0, st>>>(static_cast<const float*>(K), n, part, mt);
  else
    var_partial_kernel<__nv_bfloat16><<<dim3(mt, Hkv), KT_THREADS, 0, st>>>(static_cast<const __nv_bfloat16*>(K), n, part, mt);
  var_final_kernel<<<Hkv, FATHOM_D * VF_LANES, 0, st>>>(part, mt, n, mean, var_tmp);
  // (2) covariance partials
  int slots;
  {
    slots = (int)((n + COV_ROWS - 1) / COV_ROWS);
    const size_t smem = (size_t)FATHOM_D * PANEL * sizeof(float);
    if (k_dtype == FATHOM_F32) {
      FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(cov_partial_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      cov_partial_kernel<float><<<dim3(slots, Hkv), KT_THREADS, smem, st>>>(static_cast<const float*>(K), n, mean, pcov, slots);
    } else {
      FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(cov_partial_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
      cov_partial_kernel<__nv_bfloat16><<<dim3(slots, Hkv), KT_THREADS, smem, st>>>(static_cast<const __nv_bfloat16*>(K), n, mean, pcov, slots);
    }
  }
  // (3) partials summed in fp64 in slot order
  cov_final_kernel<<<dim3(FATHOM_D, Hkv), FATHOM_D, 0, st>>>(pcov, slots, n, cov);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_rotate_keys(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                                  const float* basis, float* K_rot, void* stream) {
  if (!ctx || !K || !mean || !basis || !K_rot) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K) || !fathom_aligned16(basis) || !fathom_aligned16(K_rot)) return FATHOM_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // tensor cores (tf32 operands split in two, three products) unless FATHOM_ROTATE_PATH=simt asks for the plain fp32 kernel
  const char* path = getenv("FATHOM_ROTATE_PATH");
  if (!(path && strcmp(path, "simt") == 0)) {
    if (fathom_rotate_tc_scratch_bytes(L->n_kv_heads) > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
    return fathom_launch_rotate_tc(ctx, L, K, k_dtype, mean, basis, K_rot, ctx->scratch, st);
  }
  const size_t smem = (size_t)2 * FATHOM_D * PANEL * sizeof(float);
  dim3 grid((unsigned)((L->n + FATHOM_D - 1) / FATHOM_D), (unsigned)L->n_kv_heads);
  if (k_dtype == FATHOM_F32) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_keys_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    rotate_keys_kernel<float><<<grid, KT_THREADS, smem, st>>>(static_cast<const float*>(K), mean, basis, K_rot, L->n);
  } else {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(rotate_keys_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    rotate_keys_kernel<__nv_bfloat16><<<grid, KT_THREADS, smem, st>>>(static_cast<const __nv_bfloat16*>(K), mean, basis, K_rot, L->n);
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_rotate_query(fathom_ctx* ctx, const fathom_layout* L, const float* q, const float* basis, float* q_rot,
                                   void* stream) {
  if (!ctx || !q || !basis || !q_rot) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  rotate_query_kernel<<<L->n_q_heads, FATHOM_D, 0, static_cast<cudaStream_t>(stream)>>>(q, basis, q_rot, L->n_q_heads / L->n_kv_heads);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_build_planes_rotated(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype, const float* mean,
                                           const float* basis, uint64_t* planes, uint16_t* scales, void* stream) {
  if (!ctx || !K || !mean || !basis || !planes || !scales) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K) || !fathom_aligned16(basis) || !fathom_aligned16(planes) || !fathom_aligned16(scales)) return FATHOM_ERR_ALIGNMENT;
  if (fathom_rotate_tc_scratch_bytes(L->n_kv_heads) > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  return fathom_launch_rotate_build_tc(ctx, L, K, k_dtype, mean, basis, planes, scales, ctx->scratch, static_cast<cudaStream_t>(stream));
}
