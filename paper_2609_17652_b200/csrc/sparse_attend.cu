// fathom_sparse_attend: gather of the selected K/V rows + exact softmax attention (Sec. 2 "Top-k decoding").
//
// Split-k: CTA (split, head) handles FATHOM_ATTN_CHUNK selected rows.  Logits and the weighted V sum both give half a warp to a row (a row is
// 256 B in bf16: 16 lanes x 16 bytes, one fully coalesced row per half-warp and load instruction), 16 rows per
// half-warp with eight in flight; the partial sums are combined in a fixed order.  Every CTA
// publishes its (max, denominator, weighted sum) triple and takes a ticket; the CTA that draws the last
// ticket of a head merges all triples in split order, so the output is bit-reproducible whichever CTA
// that is, and no second launch is needed.
#include "fathom_common.cuh"

#include <mutex>

namespace {

constexpr int AT_THREADS = FATHOM_ATTN_CHUNK;   // 128 threads: one per row, then one per channel
constexpr int AT_WARPS = AT_THREADS / 32;

// eight consecutive channels of a row, as loaded (converted to fp32 only when used, to keep many rows in flight)
struct Raw8h { uint4 x; };
struct Raw8f { float4 a, b; };
__device__ __forceinline__ Raw8h load_raw(const __nv_bfloat16* p) { Raw8h r; r.x = __ldg(reinterpret_cast<const uint4*>(p)); return r; }
__device__ __forceinline__ Raw8f load_raw(const float* p) {
  Raw8f r; r.a = __ldg(reinterpret_cast<const float4*>(p)); r.b = __ldg(reinterpret_cast<const float4*>(p) + 1); return r;
}
__device__ __forceinline__ void unpack(const Raw8h& r, float v[8]) {
  const uint32_t w[4] = {r.x.x, r.x.y, r.x.z, r.x.w};
#pragma unroll
  for (int c = 0; c < 4; ++c) { v[2 * c] = __uint_as_float(w[c] << 16); v[2 * c + 1] = __uint_as_float(w[c] & 0xffff0000u); }
}
__device__ __forceinline__ void unpack(const Raw8f& r, float v[8]) {
  v[0] = r.a.x; v[1] = r.a.y; v[2] = r.a.z; v[3] = r.a.w; v[4] = r.b.x; v[5] = r.b.y; v[6] = r.b.z; v[7] = r.b.w;
}
template <typename T> struct RawOf;
template <> struct RawOf<__nv_bfloat16> { using type = Raw8h; };
template <> struct RawOf<float> { using type = Raw8f; };
template <typename T>
__global__ void __launch_bounds__(AT_THREADS)
attend_partial_kernel(const float* __restrict__ q, const T* __restrict__ Krows, const T* __restrict__ Vrows,
                      const int32_t* __restrict__ idx, int k, long long n, int G, float softmax_scale,
                      float* __restrict__ partial, int splits, unsigned int* __restrict__ tickets,
                      float* __restrict__ result) {
  __shared__ float s_q[FATHOM_D];
  __shared__ float s_p[AT_THREADS];
  __shared__ int32_t s_idx[AT_THREADS];
  __shared__ float s_red[AT_WARPS];
  __shared__ float s_acc[AT_THREADS / 16][FATHOM_D];          // one partial sum per half-warp
  const int split = blockIdx.x, head = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kv = head / G;
  FATHOM_PDL_WAIT();                                          // the indices come from the previous kernel
  const T* Kh = Krows + (size_t)kv * (size_t)n * FATHOM_D;
  const T* Vh = Vrows + (size_t)kv * (size_t)n * FATHOM_D;
  s_q[tid] = q[(size_t)head * FATHOM_D + tid];
  const int pos = split * AT_THREADS + tid;
  const bool valid = pos < k;
  int32_t row = 0;
  if (valid) {
    row = idx[(size_t)head * k + pos];
    row = (row < 0) ? 0 : ((long long)row >= n ? (int32_t)(n - 1) : row);   // out-of-range indices are clamped, never dereferenced
  }
  s_idx[tid] = row;
  __syncthreads();

  // Half a warp per row (16 lanes x 8 channels = one fully coalesced row per load instruction), 16 rows per half-warp.
  // All 16 K rows of the half-warp are requested at once; its 16 V rows are requested as soon as the K rows have been
  // used, so that they arrive while the chunk maximum and the exponentials are computed.
  using Raw = typename RawOf<T>::type;
  const int hw = tid >> 4, l16 = tid & 15;
  Raw raw[16];
#pragma unroll
  for (int u = 0; u < 16; ++u) raw[u] = load_raw(Kh + (size_t)s_idx[hw * 16 + u] * FATHOM_D + l16 * 8);
  {
    float qv[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) qv[c] = s_q[l16 * 8 + c];
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      float x[8];
      unpack(raw[u], x);
      float part = 0.0f;
#pragma unroll
      for (int c = 0; c < 8; ++c) part = fmaf(x[c], qv[c], part);
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);   // fixed butterfly order
      if (l16 == 0) s_p[hw * 16 + u] = part;
    }
  }
#pragma unroll
  for (int u = 0; u < 16; ++u) raw[u] = load_raw(Vh + (size_t)s_idx[hw * 16 + u] * FATHOM_D + l16 * 8);
  __syncthreads();
  const float e = valid ? s_p[tid] * softmax_scale : -INFINITY;
  __syncthreads();                                           // s_p is reused for the probabilities below
  float m = e;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) s_red[warp] = m;
  __syncthreads();
  m = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
  const float p = valid ? expf(e - m) : 0.0f;
  s_p[tid] = p;
  float l = p;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  __syncthreads();                                           // s_red reads done, s_p visible
  if (lane == 0) s_red[warp] = l;

  // weighted V sum (lane = 8 channels); the eight half-warps are summed in a fixed order
  {
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      float x[8];
      unpack(raw[u], x);
      const float pr = s_p[hw * 16 + u];                       // rows past k carry probability 0
#pragma unroll
      for (int c = 0; c < 8; ++c) acc[c] = fmaf(pr, x[c], acc[c]);
    }
#pragma unroll
    for (int c = 0; c < 8; ++c) s_acc[hw][l16 * 8 + c] = acc[c];
  }
  __syncthreads();
  float* out = partial + ((size_t)head * splits + split) * (FATHOM_D + 2);
  out[2 + tid] = (((s_acc[0][tid] + s_acc[1][tid]) + (s_acc[2][tid] + s_acc[3][tid])) +
                  ((s_acc[4][tid] + s_acc[5][tid]) + (s_acc[6][tid] + s_acc[7][tid])));
  if (tid == 0) { out[0] = m; out[1] = ((s_red[0] + s_red[1]) + s_red[2]) + s_red[3]; }

  // ---- publish; the CTA that draws the head's last ticket merges all chunks (and re-arms the ticket counter)
  __shared__ bool s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned int t = atomicAdd(&tickets[head], 1u);
    s_last = (t == (unsigned int)splits - 1u);
    if (s_last) tickets[head] = 0u;
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* P = partial + (size_t)head * splits * (FATHOM_D + 2);
  float M = -INFINITY;
#pragma unroll 8
  for (int s = 0; s < splits; ++s) M = fmaxf(M, __ldcg(P + (size_t)s * (FATHOM_D + 2)));
  float num = 0.0f, den = 0.0f;
#pragma unroll 8
  for (int s = 0; s < splits; ++s) {
    const float* ps = P + (size_t)s * (FATHOM_D + 2);
    const float w = expf(__ldcg(ps) - M);
    den = fmaf(w, __ldcg(ps + 1), den);
    num = fmaf(w, __ldcg(ps + 2 + tid), num);
  }
  result[(size_t)head * FATHOM_D + tid] = num / den;
}

}  // namespace

extern "C" int fathom_sparse_attend(fathom_ctx* ctx, const fathom_layout* L, const float* q, const void* Krows,
                                    const void* Vrows, int row_dtype, const int32_t* idx, int k, float softmax_scale,
                                    float* out, void* stream) {
  if (!ctx || !q || !Krows || !Vrows || !idx || !out) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k < 1 || k > L->n) return FATHOM_ERR_INVALID_ARG;
  if (row_dtype != FATHOM_BF16 && row_dtype != FATHOM_F32) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(Krows) || !fathom_aligned16(Vrows)) return FATHOM_ERR_ALIGNMENT;
  const int Hq = L->n_q_heads, G = Hq / L->n_kv_heads;
  if (Hq > FATHOM_CTL_MAX_HEADS) return FATHOM_ERR_UNSUPPORTED;
  fathom_attn_scratch S = fathom_carve_attn(ctx->scratch, Hq, k);
  if (S.bytes > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  unsigned int* tickets = ctx->dev_status + FATHOM_CTL_TICKETS;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dim3 grid((unsigned)S.splits, (unsigned)Hq);
  // launched so that its CTAs may become resident while the selection kernel (one CTA per head) still runs
  if (row_dtype == FATHOM_BF16)
    FATHOM_CUDA_TRY(ctx, fathom_launch_dependent(attend_partial_kernel<__nv_bfloat16>, grid, dim3(AT_THREADS), 0, st, q,
                                                 static_cast<const __nv_bfloat16*>(Krows), static_cast<const __nv_bfloat16*>(Vrows), idx, k,
                                                 (long long)L->n, G, softmax_scale, S.partial, S.splits, tickets, out));
  else
    FATHOM_CUDA_TRY(ctx, fathom_launch_dependent(attend_partial_kernel<float>, grid, dim3(AT_THREADS), 0, st, q,
                                                 static_cast<const float*>(Krows), static_cast<const float*>(Vrows), idx, k,
                                                 (long long)L->n, G, softmax_scale, S.partial, S.splits, tickets, out));
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

// ---- allocation-free variant --------------------------------------------------------------------------
// Scratch for callers that cannot allocate: the per-chunk (max, denominator, weighted sum) triples live in
// this array instead of a context's arena.  In host code the name below is only a handle for the runtime,
// not a device address, so the address is fetched once per device with cudaGetSymbolAddress and that
// pointer is what the kernels receive.
static __device__ __align__(256) float g_attend_static_partials[FATHOM_ATTEND_STATIC_MAX_CHUNKS * (FATHOM_D + 2)];
// Ticket counters of the merge step, one per query head; zero when the library is loaded and re-armed by
// the merging CTA of every call, so they never need clearing either.
static __device__ __align__(256) unsigned int g_attend_static_tickets[FATHOM_ATTEND_STATIC_MAX_CHUNKS];

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
float* g_static_partials_ptr[STATIC_MAX_DEVICES];            // device address per device ordinal, null until first use
unsigned int* g_static_tickets_ptr[STATIC_MAX_DEVICES];
std::mutex g_static_mutex;
}  // namespace

extern "C" int fathom_sparse_attend_static(const fathom_layout* L, const float* q, const void* Krows, const void* Vrows,
                                           int row_dtype, const int32_t* idx, int k, float softmax_scale, float* out,
                                           void* stream) {
  if (!q || !Krows || !Vrows || !idx || !out) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k < 1 || k > L->n) return FATHOM_ERR_INVALID_ARG;
  if (row_dtype != FATHOM_BF16 && row_dtype != FATHOM_F32) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(Krows) || !fathom_aligned16(Vrows)) return FATHOM_ERR_ALIGNMENT;
  const int Hq = L->n_q_heads, G = Hq / L->n_kv_heads;
  const int splits = (k + FATHOM_ATTN_CHUNK - 1) / FATHOM_ATTN_CHUNK;
  if ((long long)Hq * splits > FATHOM_ATTEND_STATIC_MAX_CHUNKS) return FATHOM_ERR_STATIC_LIMIT;

  // set-up, once per device, with that device current
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return FATHOM_ERR_CUDA;
  if (dev < 0 || dev >= STATIC_MAX_DEVICES) return FATHOM_ERR_UNSUPPORTED;
  float* partial = nullptr;
  unsigned int* tickets = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_partials_ptr[dev]) {
      void *p = nullptr, *t = nullptr;
      if (cudaGetSymbolAddress(&p, g_attend_static_partials) != cudaSuccess || !p) return FATHOM_ERR_CUDA;
      if (cudaGetSymbolAddress(&t, g_attend_static_tickets) != cudaSuccess || !t) return FATHOM_ERR_CUDA;
      g_static_tickets_ptr[dev] = static_cast<unsigned int*>(t);
      g_static_partials_ptr[dev] = static_cast<float*>(p);
    }
    partial = g_static_partials_ptr[dev];
    tickets = g_static_tickets_ptr[dev];
  }

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  dim3 grid((unsigned)splits, (unsigned)Hq);
  if (row_dtype == FATHOM_BF16)
    attend_partial_kernel<__nv_bfloat16><<<grid, AT_THREADS, 0, st>>>(
        q, static_cast<const __nv_bfloat16*>(Krows), static_cast<const __nv_bfloat16*>(Vrows), idx, k, L->n, G,
        softmax_scale, partial, splits, tickets, out);
  else
    attend_partial_kernel<float><<<grid, AT_THREADS, 0, st>>>(q, static_cast<const float*>(Krows),
                                                              static_cast<const float*>(Vrows), idx, k, L->n, G,
                                                              softmax_scale, partial, splits, tickets, out);
  if (cudaGetLastError() != cudaSuccess) return FATHOM_ERR_CUDA;
  return FATHOM_OK;
}
