// fathom_build_planes: K -> channel-major bit planes + fp16 block scales (Sec. 3.2, Eq. 2).
//
// One thread owns one channel of one 64-token block: it keeps the 64 values of its column in
// registers (the 128 threads of a CTA read each token row as 512 contiguous bytes), takes the
// block maximum, rounds a/8 to fp16 and derives the four plane bits of every code by comparing k
// with exact multiples of the stored scale, most significant bit first:
//     bit0 = k >= 0;  bit1 = k >= (bit0 ? 4 : -4) s;  bit2 = k >= thr1 + (bit1 ? 2 : -2) s;  ...
// m * s (|m| <= 7, s an fp16 value) is exact in fp32, so the four comparisons give exactly
// clip(floor(k / s), -8, 7) + 8 with no division.  A CTA walks BLOCKS_PER_CTA consecutive blocks
// so that the 8-byte words it writes to one (channel, plane) row fill whole 32-byte sectors in L2.
#include "fathom_common.cuh"

namespace {

constexpr int BLOCKS_PER_CTA = 8;

__device__ __forceinline__ float load_k(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_k(const __nv_bfloat16* p) {
  return __bfloat162float(__ldg(p));
}

template <typename T>
__global__ void __launch_bounds__(FATHOM_D)
build_planes_kernel(const T* __restrict__ K, uint64_t* __restrict__ planes, uint16_t* __restrict__ scales,
                    long long n, long long nb, long long plane_stride, long long scale_stride) {
  const int j = threadIdx.x;                                  // channel
  const int h = blockIdx.y;                                   // KV head
  const long long b0 = (long long)blockIdx.x * BLOCKS_PER_CTA;
  const T* Kh = K + (size_t)h * (size_t)n * FATHOM_D;
  uint64_t* prow = planes + ((size_t)h * FATHOM_D + j) * FATHOM_NPLANES * (size_t)plane_stride;
  uint16_t* srow = scales + ((size_t)h * FATHOM_D + j) * (size_t)scale_stride;

  for (int bb = 0; bb < BLOCKS_PER_CTA; ++bb) {
    const long long b = b0 + bb;
    if (b >= nb) break;
    const long long i0 = b * FATHOM_BLOCK;
    const int valid = (int)min((long long)FATHOM_BLOCK, n - i0);

    float v[FATHOM_BLOCK];
    if (valid == FATHOM_BLOCK) {
#pragma unroll
      for (int i = 0; i < FATHOM_BLOCK; ++i) v[i] = load_k(Kh + (size_t)(i0 + i) * FATHOM_D + j);
    } else {
#pragma unroll
      for (int i = 0; i < FATHOM_BLOCK; ++i) v[i] = (i < valid) ? load_k(Kh + (size_t)(i0 + i) * FATHOM_D + j) : 0.0f;
    }
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < FATHOM_BLOCK; ++i) a = fmaxf(a, fabsf(v[i]));

    const __half sh = __float2half_rn(a * 0.125f);            // a/8 is exact; one rounding to fp16
    const float s = __half2float(sh);
    const float s2 = s * 2.0f, s4 = s * 4.0f;

    uint32_t w[FATHOM_NPLANES][2] = {{0u, 0u}, {0u, 0u}, {0u, 0u}, {0u, 0u}};
    if (s > 0.0f) {
#pragma unroll
      for (int i = 0; i < FATHOM_BLOCK; ++i) {
        const float k = v[i];
        const uint32_t m = 1u << (i & 31);
        const bool c0 = k >= 0.0f;
        float thr = c0 ? s4 : -s4;
        const bool c1 = k >= thr;
        thr += c1 ? s2 : -s2;
        const bool c2 = k >= thr;
        thr += c2 ? s : -s;
        const bool c3 = k >= thr;
        if (c0) w[0][i >> 5] |= m;
        if (c1) w[1][i >> 5] |= m;
        if (c2) w[2][i >> 5] |= m;
        if (c3) w[3][i >> 5] |= m;
      }
      if (valid < FATHOM_BLOCK) {                             // absent tail tokens carry 0 bits
        const uint64_t keep = (valid == 0) ? 0ull : (~0ull >> (64 - valid));
#pragma unroll
        for (int p = 0; p < FATHOM_NPLANES; ++p) {
          w[p][0] &= (uint32_t)keep;
          w[p][1] &= (uint32_t)(keep >> 32);
        }
      }
    } else {                                                  // zero scale: every code is 8 = 0b1000
      const uint64_t keep = ~0ull >> (64 - valid);
      w[0][0] = (uint32_t)keep;
      w[0][1] = (uint32_t)(keep >> 32);
    }
#pragma unroll
    for (int p = 0; p < FATHOM_NPLANES; ++p)
      prow[(size_t)p * plane_stride + b] = ((uint64_t)w[p][1] << 32) | w[p][0];
    srow[b] = __half_as_ushort(sh);
  }
}

}  // namespace

extern "C" int fathom_build_planes(fathom_ctx* ctx, const fathom_layout* L, const void* K, int k_dtype,
                                   uint64_t* planes, uint16_t* scales, void* stream) {
  if (!ctx || !K || !planes || !scales) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k_dtype != FATHOM_F32 && k_dtype != FATHOM_BF16) return FATHOM_ERR_UNSUPPORTED;
  if (!fathom_aligned16(K) || !fathom_aligned16(planes) || !fathom_aligned16(scales)) return FATHOM_ERR_ALIGNMENT;
  const long long nb = fathom_nblocks(L->n);
  dim3 grid((unsigned)((nb + BLOCKS_PER_CTA - 1) / BLOCKS_PER_CTA), (unsigned)L->n_kv_heads);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (k_dtype == FATHOM_F32)
    build_planes_kernel<float><<<grid, FATHOM_D, 0, st>>>(static_cast<const float*>(K), planes, scales, L->n, nb,
                                                         L->plane_stride_words, L->scale_stride);
  else
    build_planes_kernel<__nv_bfloat16><<<grid, FATHOM_D, 0, st>>>(static_cast<const __nv_bfloat16*>(K), planes, scales,
                                                                 L->n, nb, L->plane_stride_words, L->scale_stride);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
