// fathom_build_planes: K -> channel-major bit planes + fp16 block scales (Sec. 3.2, Eq. 2).
//
// Two threads own one channel of a 64-token block (32 tokens each): the 128 threads of a token half read
// every token row as 512 contiguous bytes, keep their 32 values in registers, exchange the two half maxima
// through shared memory, round a/8 to fp16 and derive the four plane bits of every code by comparing k
// with exact multiples of the stored scale, most significant bit first:
//     bit0 = k >= 0;  bit1 = k >= (bit0 ? 4 : -4) s;  bit2 = k >= thr1 + (bit1 ? 2 : -2) s;  ...
// m * s (|m| <= 7, s an fp16 value) is exact in fp32, so the four comparisons give exactly
// clip(floor(k / s), -8, 7) + 8 with no division.  A CTA walks BLOCKS_PER_CTA consecutive blocks and
// collects their plane words and scales in shared memory, then writes every (channel, plane) row segment
// as whole 32-byte sectors (partial-sector writes cost a fill read each).
#include "fathom_common.cuh"

namespace {

constexpr int BP_THREADS = 2 * FATHOM_D;
constexpr int BLOCKS_PER_CTA = 8;
constexpr int HALF = FATHOM_BLOCK / 2;                         // tokens per thread
constexpr int OUT_PITCH = FATHOM_NPLANES * BLOCKS_PER_CTA * 2 + 1;

__device__ __forceinline__ float load_k(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_k(const __nv_bfloat16* p) { return __bfloat162float(__ldg(p)); }

template <typename T>
__global__ void __launch_bounds__(BP_THREADS)
build_planes_kernel(const T* __restrict__ K, uint32_t* __restrict__ planes32, uint16_t* __restrict__ scales,
                    long long n, long long nb, long long plane_stride, long long scale_stride) {
  __shared__ float s_amax[2][2][FATHOM_D];                     // [parity of block][token half][channel]
  __shared__ uint32_t s_out[FATHOM_D][OUT_PITCH];              // [channel][plane][block][half], padded against bank conflicts
  __shared__ uint16_t s_scale[FATHOM_D][BLOCKS_PER_CTA];
  const int j = threadIdx.x & (FATHOM_D - 1);                  // channel
  const int half = threadIdx.x >> 7;                           // 0: tokens 0..31 of the block, 1: tokens 32..63
  const int h = blockIdx.y;                                    // KV head
  const long long b0 = (long long)blockIdx.x * BLOCKS_PER_CTA;
  const T* Kh = K + (size_t)h * (size_t)n * FATHOM_D;

  for (int bb = 0; bb < BLOCKS_PER_CTA; ++bb) {
    const long long b = b0 + bb;
    if (b >= nb) break;                                        // uniform over the CTA
    const long long i0 = b * FATHOM_BLOCK + half * HALF;
    const int valid = (int)min((long long)HALF, n - i0);       // of this thread's 32 tokens (may be <= 0)

    float v[HALF];
    if (valid >= HALF) {
#pragma unroll
      for (int i = 0; i < HALF; ++i) v[i] = load_k(Kh + (size_t)(i0 + i) * FATHOM_D + j);
    } else {
#pragma unroll
      for (int i = 0; i < HALF; ++i) v[i] = (i < valid) ? load_k(Kh + (size_t)(i0 + i) * FATHOM_D + j) : 0.0f;
    }
    float a = 0.0f;
#pragma unroll
    for (int i = 0; i < HALF; ++i) a = fmaxf(a, fabsf(v[i]));
    s_amax[bb & 1][half][j] = a;
    __syncthreads();
    a = fmaxf(a, s_amax[bb & 1][half ^ 1][j]);

    const __half sh = __float2half_rn(a * 0.125f);             // a/8 is exact; one rounding to fp16
    const float sc = __half2float(sh);
    const float s2 = sc * 2.0f, s4 = sc * 4.0f;

    uint32_t w[FATHOM_NPLANES] = {0u, 0u, 0u, 0u};
    const uint32_t keep = (valid >= HALF) ? ~0u : (valid <= 0 ? 0u : (~0u >> (32 - valid)));   // absent tail tokens carry 0 bits
    if (sc > 0.0f) {
#pragma unroll
      for (int i = 0; i < HALF; ++i) {
        const float k = v[i];
        const uint32_t m = 1u << i;
        const bool c0 = k >= 0.0f;
        float thr = c0 ? s4 : -s4;
        const bool c1 = k >= thr;
        thr += c1 ? s2 : -s2;
        const bool c2 = k >= thr;
        thr += c2 ? sc : -sc;
        const bool c3 = k >= thr;
        if (c0) w[0] |= m;
        if (c1) w[1] |= m;
        if (c2) w[2] |= m;
        if (c3) w[3] |= m;
      }
#pragma unroll
      for (int p = 0; p < FATHOM_NPLANES; ++p) w[p] &= keep;
    } else {                                                   // zero scale: every code is 8 = 0b1000
      w[0] = keep;
    }
    // little-endian halves of the 64-bit plane word: tokens 0..31 in the low 32 bits
#pragma unroll
    for (int p = 0; p < FATHOM_NPLANES; ++p) s_out[j][(p * BLOCKS_PER_CTA + bb) * 2 + half] = w[p];
    if (half == 0) s_scale[j][bb] = __half_as_ushort(sh);
  }
  __syncthreads();

  // ---- flush: each (channel, plane) row segment is BLOCKS_PER_CTA words = 64 contiguous bytes
  const int nblk = (int)min((long long)BLOCKS_PER_CTA, nb - b0);
  uint64_t* planes64 = reinterpret_cast<uint64_t*>(planes32);
  for (int e = threadIdx.x; e < FATHOM_D * FATHOM_NPLANES * (BLOCKS_PER_CTA / 2); e += BP_THREADS) {
    const int pair = e % (BLOCKS_PER_CTA / 2);                 // two words = one 16-byte store
    const int p = (e / (BLOCKS_PER_CTA / 2)) % FATHOM_NPLANES;
    const int c = e / (BLOCKS_PER_CTA / 2 * FATHOM_NPLANES);
    const uint32_t* src = &s_out[c][(p * BLOCKS_PER_CTA + 2 * pair) * 2];
    uint64_t* dst = planes64 + (((size_t)h * FATHOM_D + c) * FATHOM_NPLANES + p) * (size_t)plane_stride + b0 + 2 * pair;
    if (2 * pair + 1 < nblk) {
      *reinterpret_cast<uint4*>(dst) = make_uint4(src[0], src[1], src[2], src[3]);
    } else if (2 * pair < nblk) {
      dst[0] = ((uint64_t)src[1] << 32) | src[0];
    }
  }
  for (int e = threadIdx.x; e < FATHOM_D; e += BP_THREADS) {
    uint16_t* dst = scales + ((size_t)h * FATHOM_D + e) * (size_t)scale_stride + b0;
    if (nblk == BLOCKS_PER_CTA) {
      const uint16_t* sp = s_scale[e];
      *reinterpret_cast<uint4*>(dst) = make_uint4(sp[0] | ((uint32_t)sp[1] << 16), sp[2] | ((uint32_t)sp[3] << 16),
                                                  sp[4] | ((uint32_t)sp[5] << 16), sp[6] | ((uint32_t)sp[7] << 16));
    } else {
      for (int x = 0; x < nblk; ++x) dst[x] = s_scale[e][x];
    }
  }
}

template <typename T>
int launch_build(fathom_ctx* ctx, const fathom_layout* L, const T* K, uint64_t* planes, uint16_t* scales,
                 cudaStream_t st) {
  const long long nb = fathom_nblocks(L->n);
  dim3 grid((unsigned)((nb + BLOCKS_PER_CTA - 1) / BLOCKS_PER_CTA), (unsigned)L->n_kv_heads);
  build_planes_kernel<T><<<grid, BP_THREADS, 0, st>>>(K, reinterpret_cast<uint32_t*>(planes), scales, L->n, nb,
                                                      L->plane_stride_words, L->scale_stride);
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
