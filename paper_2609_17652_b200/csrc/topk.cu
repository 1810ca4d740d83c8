// fathom_topk: per-query-head top-k over n scores with deterministic ties (Sec. 2 "Top-k decoding").
//
// Bucket select on the order-preserving integer image of the fp32 score (-0 folded onto +0):
//   1. histogram of the 12 leading key bits over all eligible tokens (one read of the scores);
//   2. per head, the threshold bin b* whose suffix count first reaches the number wanted;
//   3. filter (second read): tokens in bins above b* are winners, tokens in b* are candidates;
//      both are appended with warp-aggregated atomics (ballot + popc), order irrelevant;
//   4. per head, an 8-bit radix select over the candidates on the 64-bit composite
//      (key << 32 | ~index), which makes every element distinct and encodes "ties go to the lower
//      token index"; the chosen candidates join the winners, the forced sink/local tokens are
//      added and the k indices are sorted ascending in shared memory (bitonic network).
// The set is unique, so the arbitrary append order never shows in the output.
#include "fathom_common.cuh"

namespace {

constexpr int TK_THREADS = 256;
constexpr int TK_PER_THREAD = 16;                            // 4 x float4
constexpr int TK_TILE = TK_THREADS * TK_PER_THREAD;          // 4096 scores per CTA
constexpr int FIN_THREADS = 1024;

__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u << 1) == 0u) u = 0u;                                // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Forced { long long sink_end, local_begin; };          // eligible tokens: sink_end <= i < local_begin

__global__ void __launch_bounds__(TK_THREADS)
topk_hist_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                 uint32_t* __restrict__ hist) {
  __shared__ uint32_t sh[FATHOM_TOPK_BINS];
  const int head = blockIdx.y;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += TK_THREADS) sh[b] = 0u;
  __syncthreads();
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const long long base = (long long)blockIdx.x * TK_TILE;
#pragma unroll
  for (int v = 0; v < TK_PER_THREAD / 4; ++v) {
    const long long i = base + ((long long)v * TK_THREADS + threadIdx.x) * 4;
    if (i < n) {                                             // score_stride is a multiple of 4: the float4 stays in the row
      const float4 x = __ldg(reinterpret_cast<const float4*>(row + i));
      const float e[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const long long t = i + c;
        if (t >= F.sink_end && t < F.local_begin) atomicAdd(&sh[ordered_key(e[c]) >> 20], 1u);
      }
    }
  }
  __syncthreads();
  uint32_t* g = hist + (size_t)head * FATHOM_TOPK_BINS;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += TK_THREADS) {
    const uint32_t c = sh[b];
    if (c) atomicAdd(&g[b], c);
  }
}

// state[head][0] = threshold bin, [1] = tokens in bins above it, [2] = tokens still needed from it
__global__ void __launch_bounds__(FIN_THREADS)
topk_find_bin_kernel(const uint32_t* __restrict__ hist, uint32_t* __restrict__ state, uint32_t want,
                     uint32_t* __restrict__ dev_status) {
  __shared__ uint32_t warp_sum[32];
  const int head = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t* h = hist + (size_t)head * FATHOM_TOPK_BINS;
  // thread t owns bins 4095 - 4t .. 4092 - 4t (descending), so an inclusive scan over threads is a suffix count
  uint32_t c[4], local = 0;
#pragma unroll
  for (int x = 0; x < 4; ++x) { c[x] = h[FATHOM_TOPK_BINS - 1 - (4 * tid + x)]; local += c[x]; }
  uint32_t incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) warp_sum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = warp_sum[lane], wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    warp_sum[lane] = wi - w;                                  // exclusive
  }
  __syncthreads();
  const uint32_t above = warp_sum[warp] + incl - local;       // tokens in bins above this thread's four
  if (want == 0) {
    if (tid == 0) { state[head * 8 + 0] = FATHOM_TOPK_BINS; state[head * 8 + 1] = 0; state[head * 8 + 2] = 0; }
    return;
  }
  if (above < want && above + local >= want) {
    uint32_t run = above;
#pragma unroll
    for (int x = 0; x < 4; ++x) {
      if (run < want && run + c[x] >= want) {
        state[head * 8 + 0] = (uint32_t)(FATHOM_TOPK_BINS - 1 - (4 * tid + x));
        state[head * 8 + 1] = run;
        state[head * 8 + 2] = want - run;
      }
      run += c[x];
    }
  }
  if (tid == FIN_THREADS - 1 && above + local < want) {       // fewer eligible tokens than wanted
    atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
    state[head * 8 + 0] = 0; state[head * 8 + 1] = above + local - c[3]; state[head * 8 + 2] = c[3];
  }
}

__global__ void __launch_bounds__(TK_THREADS)
topk_filter_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   uint32_t* __restrict__ state, int32_t* __restrict__ cand, int32_t* __restrict__ winners, int k) {
  const int head = blockIdx.y, lane = threadIdx.x & 31;
  const uint32_t bstar = state[head * 8 + 0];
  const float* row = scores + (size_t)head * (size_t)score_stride;
  int32_t* cand_h = cand + (size_t)head * (size_t)n;
  int32_t* win_h = winners + (size_t)head * (size_t)k;
  const long long base = (long long)blockIdx.x * TK_TILE;
#pragma unroll
  for (int v = 0; v < TK_PER_THREAD / 4; ++v) {
    const long long i = base + ((long long)v * TK_THREADS + threadIdx.x) * 4;
    float e[4] = {0.f, 0.f, 0.f, 0.f};
    if (i < n) {
      const float4 x = __ldg(reinterpret_cast<const float4*>(row + i));
      e[0] = x.x; e[1] = x.y; e[2] = x.z; e[3] = x.w;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const long long t = i + c;
      const bool elig = t < n && t >= F.sink_end && t < F.local_begin;
      const uint32_t bin = ordered_key(e[c]) >> 20;
      const bool is_win = elig && bin > bstar;
      const bool is_cand = elig && bin == bstar;
      const unsigned mw = __ballot_sync(0xffffffffu, is_win);
      const unsigned mc = __ballot_sync(0xffffffffu, is_cand);
      if (mw) {
        uint32_t pos = 0;
        if (lane == __ffs(mw) - 1) pos = atomicAdd(&state[head * 8 + 3], (uint32_t)__popc(mw));
        pos = __shfl_sync(0xffffffffu, pos, __ffs(mw) - 1);
        if (is_win) win_h[pos + __popc(mw & ((1u << lane) - 1u))] = (int32_t)t;
      }
      if (mc) {
        uint32_t pos = 0;
        if (lane == __ffs(mc) - 1) pos = atomicAdd(&state[head * 8 + 4], (uint32_t)__popc(mc));
        pos = __shfl_sync(0xffffffffu, pos, __ffs(mc) - 1);
        if (is_cand) cand_h[pos + __popc(mc & ((1u << lane) - 1u))] = (int32_t)t;
      }
    }
  }
}

// low 52 bits of (key << 32 | ~index); the 12 leading key bits are the same for every candidate
__device__ __forceinline__ uint64_t composite52(const float* row, int32_t i) {
  return ((((uint64_t)ordered_key(row[i])) << 32) | (uint32_t)(~(uint32_t)i)) & ((1ull << 52) - 1ull);
}

__global__ void __launch_bounds__(FIN_THREADS)
topk_finish_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   uint32_t* __restrict__ state, const int32_t* __restrict__ cand, int32_t* __restrict__ winners,
                   int k, int sort_len, int32_t* __restrict__ idx_out) {
  extern __shared__ int32_t s_sort[];                         // sort_len entries
  __shared__ uint32_t s_hist[256];
  __shared__ uint64_t s_prefix;                               // chosen leading bits of the threshold composite
  __shared__ uint32_t s_need, s_digit, s_wpos;
  const int head = blockIdx.x, tid = threadIdx.x;
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const int32_t* cand_h = cand + (size_t)head * (size_t)n;
  int32_t* win_h = winners + (size_t)head * (size_t)k;
  const uint32_t m = state[head * 8 + 4];
  const uint32_t c_hi = state[head * 8 + 1];
  const uint32_t need0 = state[head * 8 + 2];

  // ---- radix select of the need0 largest composites among the m candidates.  The 12 leading key bits are
  //      equal for all of them; digits of 8 bits are taken from bit 52 downwards (the first covers 4 bits).
  uint64_t thr = 0;                                           // winners are candidates with composite >= thr
  if (need0 > 0 && need0 < m) {
    if (tid == 0) { s_prefix = 0; s_need = need0; }
    __syncthreads();
    int hi = 52;                                              // bits [hi, 64) are decided
    while (hi > 0) {
      const int bits = (hi % 8) ? (hi % 8) : 8;
      const int lo = hi - bits;
      if (tid < 256) s_hist[tid] = 0u;
      __syncthreads();
      const uint64_t prefix = s_prefix;
      for (uint32_t c = tid; c < m; c += FIN_THREADS) {
        const uint64_t comp = composite52(row, cand_h[c]);
        const bool match = (comp >> hi) == (prefix >> hi);
        if (match) atomicAdd(&s_hist[(uint32_t)(comp >> lo) & ((1u << bits) - 1u)], 1u);
      }
      __syncthreads();
      if (tid < 32) {                                         // warp 0: suffix counts over the 256 digits
        uint32_t cnt[8], local = 0;
#pragma unroll
        for (int x = 0; x < 8; ++x) { cnt[x] = s_hist[255 - (8 * tid + x)]; local += cnt[x]; }
        uint32_t incl = local;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
          if (tid >= o) incl += y;
        }
        const uint32_t need = s_need;
        uint32_t run = incl - local;
        if (run < need && run + local >= need) {
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            if (run < need && run + cnt[x] >= need) { s_digit = 255 - (8 * tid + x); s_wpos = need - run; }
            run += cnt[x];
          }
        }
      }
      __syncthreads();
      if (tid == 0) {
        s_prefix |= (uint64_t)s_digit << lo;
        s_need = s_wpos;                                      // still needed from inside the chosen digit
      }
      __syncthreads();
      hi = lo;
    }
    // composites are distinct, so exactly one candidate equals the decided low 52 bits: it is the threshold
    thr = s_prefix;
  }
  if (tid == 0) s_wpos = 0;
  __syncthreads();
  if (need0 > 0) {
    for (uint32_t c = tid; c < m; c += FIN_THREADS) {
      const int32_t i = cand_h[c];
      const bool take = (need0 >= m) || (composite52(row, i) >= thr);
      if (take) {
        const uint32_t pos = atomicAdd(&s_wpos, 1u);
        if (c_hi + pos < (uint32_t)k) win_h[c_hi + pos] = i;
      }
    }
  }
  __syncthreads();

  // ---- gather forced tokens + winners, sort ascending, write
  const int n_sink = (int)F.sink_end;
  const int n_loc = (int)(n - F.local_begin);
  const int n_forced = n_sink + n_loc;
  const int n_win = min((int)(c_hi + s_wpos), k - n_forced);
  for (int e = tid; e < sort_len; e += FIN_THREADS) {
    int32_t v = 0x7fffffff;
    if (e < n_sink) v = e;
    else if (e < n_forced) v = (int32_t)(F.local_begin + (e - n_sink));
    else if (e < n_forced + n_win) v = win_h[e - n_forced];
    s_sort[e] = v;
  }
  __syncthreads();
  for (int size = 2; size <= sort_len; size <<= 1) {
    for (int stride = size >> 1; stride > 0; stride >>= 1) {
      for (int e = tid; e < sort_len / 2; e += FIN_THREADS) {
        const int lo_i = 2 * e - (e & (stride - 1));
        const int hi_i = lo_i + stride;
        const bool up = (lo_i & size) == 0;
        const int32_t a = s_sort[lo_i], b = s_sort[hi_i];
        if ((a > b) == up) { s_sort[lo_i] = b; s_sort[hi_i] = a; }
      }
      __syncthreads();
    }
  }
  for (int e = tid; e < k; e += FIN_THREADS) idx_out[(size_t)head * k + e] = s_sort[e];
}

}  // namespace

extern "C" int fathom_topk(fathom_ctx* ctx, const fathom_layout* L, const float* scores, int k, int n_sink,
                           int n_local, int32_t* idx, void* stream) {
  if (!ctx || !scores || !idx) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  if (k < 1 || k > L->n || k > FATHOM_MAX_K || n_sink < 0 || n_local < 0) return FATHOM_ERR_INVALID_ARG;
  if (!fathom_aligned16(scores)) return FATHOM_ERR_ALIGNMENT;
  const long long n = L->n;
  Forced F;
  F.sink_end = n_sink < n ? n_sink : n;
  F.local_begin = (n - n_local > F.sink_end) ? (n - n_local) : F.sink_end;
  const long long n_forced = F.sink_end + (n - F.local_begin);
  if (n_forced > k) return FATHOM_ERR_INVALID_ARG;
  const int Hq = L->n_q_heads;
  fathom_topk_scratch S = fathom_carve_topk(ctx->scratch, Hq, n, k);
  if (S.bytes > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint32_t want = (uint32_t)(k - n_forced);

  // histograms and per-head state are contiguous at the start of the arena
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.cand - (char*)S.hist, st));
  dim3 grid((unsigned)((n + TK_TILE - 1) / TK_TILE), (unsigned)Hq);
  topk_hist_kernel<<<grid, TK_THREADS, 0, st>>>(scores, n, L->score_stride, F, S.hist);
  topk_find_bin_kernel<<<Hq, FIN_THREADS, 0, st>>>(S.hist, S.state, want, ctx->dev_status);
  topk_filter_kernel<<<grid, TK_THREADS, 0, st>>>(scores, n, L->score_stride, F, S.state, S.cand, S.winners, k);
  int sort_len = 2;
  while (sort_len < k) sort_len <<= 1;
  const size_t smem = (size_t)sort_len * sizeof(int32_t);
  if (smem > 48 * 1024)
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(topk_finish_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  topk_finish_kernel<<<Hq, FIN_THREADS, smem, st>>>(scores, n, L->score_stride, F, S.state, S.cand, S.winners, k,
                                                    sort_len, idx);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
