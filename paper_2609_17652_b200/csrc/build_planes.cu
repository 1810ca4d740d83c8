// fathom_build_planes: K -> channel-major bit planes + fp16 block scales (Sec. 3.2, Eq. 2).
//
// A 64-token block of one KV head is 64 x 128 contiguous values (32 KB in fp32), so it is fetched with
// one bulk asynchronous copy (cp.async.bulk, global -> shared, completion on an mbarrier) into a
// STAGES-deep ring; persistent CTAs walk contiguous runs of blocks so that loads for the next blocks
// are in flight while the current one is quantised.  One thread owns one channel: it pulls its column
// out of shared memory (bank = channel mod 32, conflict-free), takes the block maximum, rounds a/8 to
// fp16 and derives the four plane bits of every code by comparing k with exact multiples of the
// stored scale, most significant bit first:
//     bit0 = k >= 0;  bit1 = k >= (bit0 ? 4 : -4) s;  bit2 = k >= thr1 + (bit1 ? 2 : -2) s;  ...
// m * s (|m| <= 7, s an fp16 value) is exact in fp32, so the four comparisons give exactly
// clip(floor(k / s), -8, 7) + 8 with no division.  Consecutive blocks of a CTA write consecutive
// 8-byte words of each (channel, plane) row, which merge into full sectors in L2.
#include "fathom_common.cuh"

namespace {

constexpr int STAGES = 3;
constexpr uint32_t WAIT_LIMIT = 1u << 24;                     // bounded spin on the load barrier

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Returns false when the wait gave up (the caller records it and leaves).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  for (uint32_t it = 0; it < WAIT_LIMIT; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__global__ void __launch_bounds__(FATHOM_D, 2)
build_planes_kernel(const T* __restrict__ K, uint64_t* __restrict__ planes, uint16_t* __restrict__ scales,
                    long long n, long long nb, long long plane_stride, long long scale_stride,
                    long long total_blocks, long long chunk, uint32_t* __restrict__ dev_status) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t full[STAGES];
  T* tiles = reinterpret_cast<T*>(smem_raw);                   // [STAGES][64][128]
  constexpr uint32_t ROW_BYTES = FATHOM_D * sizeof(T);
  constexpr int TILE_ELEMS = FATHOM_BLOCK * FATHOM_D;

  const int j = threadIdx.x;                                   // channel
  const long long first = (long long)blockIdx.x * chunk;
  const long long count = min(chunk, total_blocks - first);
  if (count <= 0) return;

  if (j == 0) {
    for (int s = 0; s < STAGES; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  auto issue = [&](long long s) {                              // thread 0 only
    const long long gb = first + s;
    const long long h = gb / nb, b = gb % nb;
    const uint32_t valid = (uint32_t)min((long long)FATHOM_BLOCK, n - b * FATHOM_BLOCK);
    const int st = (int)(s % STAGES);
    mbar_expect_tx(&full[st], valid * ROW_BYTES);
    bulk_load(tiles + (size_t)st * TILE_ELEMS, K + ((size_t)h * (size_t)n + (size_t)b * FATHOM_BLOCK) * FATHOM_D,
              valid * ROW_BYTES, &full[st]);
  };
  if (j == 0)
    for (long long s = 0; s < min((long long)STAGES, count); ++s) issue(s);

  for (long long s = 0; s < count; ++s) {
    const long long gb = first + s;
    const long long h = gb / nb, b = gb % nb;
    const int valid = (int)min((long long)FATHOM_BLOCK, n - b * FATHOM_BLOCK);
    const int st = (int)(s % STAGES);
    if (!mbar_wait_bounded(&full[st], (uint32_t)((s / STAGES) & 1))) {
      if (j == 0) atomicOr(dev_status, FATHOM_DEV_WAIT_EXPIRED);
      // give the copies still in flight a bounded chance to land before this CTA's shared memory is released
      for (int q = 0; q < STAGES; ++q) mbar_wait_bounded(&full[q], (uint32_t)(((s + q) / STAGES) & 1));
      return;
    }
    const T* tile = tiles + (size_t)st * TILE_ELEMS;
    float v[FATHOM_BLOCK];
#pragma unroll
    for (int i = 0; i < FATHOM_BLOCK; ++i) v[i] = to_f32(tile[i * FATHOM_D + j]);
    __syncthreads();                                           // every thread has its column: the stage is free
    if (j == 0 && s + STAGES < count) issue(s + STAGES);
    if (valid < FATHOM_BLOCK) {
#pragma unroll
      for (int i = 0; i < FATHOM_BLOCK; ++i) v[i] = (i < valid) ? v[i] : 0.0f;
    }

    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < FATHOM_BLOCK; ++i) a = fmaxf(a, fabsf(v[i]));
    const __half sh = __float2half_rn(a * 0.125f);             // a/8 is exact; one rounding to fp16
    const float sc = __half2float(sh);
    const float s2 = sc * 2.0f, s4 = sc * 4.0f;

    uint32_t w[FATHOM_NPLANES][2] = {{0u, 0u}, {0u, 0u}, {0u, 0u}, {0u, 0u}};
    const uint64_t keep = ~0ull >> (64 - valid);               // absent tail tokens carry 0 bits
    if (sc > 0.0f) {
#pragma unroll
      for (int i = 0; i < FATHOM_BLOCK; ++i) {
        const float k = v[i];
        const uint32_t m = 1u << (i & 31);
        const bool c0 = k >= 0.0f;
        float thr = c0 ? s4 : -s4;
        const bool c1 = k >= thr;
        thr += c1 ? s2 : -s2;
        const bool c2 = k >= thr;
        thr += c2 ? sc : -sc;
        const bool c3 = k >= thr;
        if (c0) w[0][i >> 5] |= m;
        if (c1) w[1][i >> 5] |= m;
        if (c2) w[2][i >> 5] |= m;
        if (c3) w[3][i >> 5] |= m;
      }
#pragma unroll
      for (int p = 0; p < FATHOM_NPLANES; ++p) {
        w[p][0] &= (uint32_t)keep;
        w[p][1] &= (uint32_t)(keep >> 32);
      }
    } else {                                                   // zero scale: every code is 8 = 0b1000
      w[0][0] = (uint32_t)keep;
      w[0][1] = (uint32_t)(keep >> 32);
    }
    uint64_t* prow = planes + (((size_t)h * FATHOM_D + j) * FATHOM_NPLANES) * (size_t)plane_stride + b;
#pragma unroll
    for (int p = 0; p < FATHOM_NPLANES; ++p)
      prow[(size_t)p * plane_stride] = ((uint64_t)w[p][1] << 32) | w[p][0];
    scales[((size_t)h * FATHOM_D + j) * (size_t)scale_stride + b] = __half_as_ushort(sh);
  }
}

template <typename T>
int launch_build(fathom_ctx* ctx, const fathom_layout* L, const T* K, uint64_t* planes, uint16_t* scales,
                 cudaStream_t st) {
  const long long nb = fathom_nblocks(L->n);
  const long long total = nb * L->n_kv_heads;
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, ctx->device);
  const long long max_ctas = 2LL * sms;                        // two resident CTAs per SM, persistent
  long long chunk = (total + max_ctas - 1) / max_ctas;
  chunk = (chunk + 7) / 8 * 8;                                 // runs of >= 8 blocks: 64-byte write segments per row
  const long long ctas = (total + chunk - 1) / chunk;
  const size_t smem = (size_t)STAGES * FATHOM_BLOCK * FATHOM_D * sizeof(T);
  FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(build_planes_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  build_planes_kernel<T><<<(unsigned)ctas, FATHOM_D, smem, st>>>(K, planes, scales, L->n, nb, L->plane_stride_words,
                                                                L->scale_stride, total, chunk, ctx->dev_status);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

}  // namespace

extern "C" int fathom_build_planes(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype,
                                   uint64_t* planes, uint16_t* scales, void* stream) {
  if (!ctx || !K || !planes || !scales) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K) || !fathom_aligned16(planes) || !fathom_aligned16(scales)) return FATHOM_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (k_dtype == FATHOM_F32) return launch_build<float>(ctx, L, static_cast<const float*>(K), planes, scales, st);
  return launch_build<__nv_bfloat16>(ctx, L, static_cast<const __nv_bfloat16*>(K), planes, scales, st);
}
