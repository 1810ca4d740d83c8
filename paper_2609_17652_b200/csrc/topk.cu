// fathom_topk: per-query-head top-k over n scores with deterministic ties (Sec. 2 "Top-k decoding").
//
// Bucket select on the order-preserving integer image of the fp32 score (-0 folded onto +0):
//   1. histogram of the 12 leading key bits over all eligible tokens (one read of the scores);
//   2. per head, the threshold bin b* whose suffix count first reaches the number wanted;
//   3. filter (second read): a lane owns one token, so the warp ballot of "bin above b*" IS the 32-token
//      word of a selection bitmap, written without atomics; tokens in bin b* itself are candidates,
//      appended with warp-aggregated atomics (ballot + popc), order irrelevant;
//   4. per head, a radix select over the candidates on the 64-bit composite (key << 32 | ~index), which
//      makes every element distinct and encodes "ties go to the lower token index"; the chosen
//      candidates and the forced sink/local tokens are OR-ed into the bitmap, and the k indices are
//      emitted in ascending order by a popcount prefix sum over the bitmap words.
// The selected set is unique, so neither the append order nor atomics can show in the output.
#include "fathom_common.cuh"

namespace {

constexpr int HIST_THREADS = 256;
constexpr int HIST_TILE = 32768;                             // scores per CTA of the histogram pass
constexpr int FILT_THREADS = 256;
constexpr int FILT_WARP_TOKENS = 1024;                       // 32 ballots -> 32 bitmap words per warp
constexpr int FILT_TILE = (FILT_THREADS / 32) * FILT_WARP_TOKENS;   // 8192 tokens per CTA
constexpr int FIN_THREADS = 1024;
constexpr int FIN_CACHE = 4096;                              // candidate composites kept in shared memory

__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u << 1) == 0u) u = 0u;                                // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

struct Forced { long long sink_end, local_begin; };          // eligible tokens: sink_end <= i < local_begin

__global__ void __launch_bounds__(HIST_THREADS)
topk_hist_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                 uint32_t* __restrict__ hist) {
  __shared__ uint32_t sh[FATHOM_TOPK_BINS];
  const int head = blockIdx.y;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += HIST_THREADS) sh[b] = 0u;
  __syncthreads();
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const long long base = (long long)blockIdx.x * HIST_TILE;
  const long long end = min(base + HIST_TILE, n);
#pragma unroll 4
  for (long long i = base + (long long)threadIdx.x * 4; i < end; i += HIST_THREADS * 4) {
    // score_stride is a multiple of 4, so the float4 stays inside the row even when it straddles n
    const float4 x = __ldg(reinterpret_cast<const float4*>(row + i));
    const float e[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const long long t = i + c;
      if (t >= F.sink_end && t < F.local_begin) atomicAdd(&sh[ordered_key(e[c]) >> 20], 1u);
    }
  }
  __syncthreads();
  uint32_t* g = hist + (size_t)head * FATHOM_TOPK_BINS;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += HIST_THREADS) {
    const uint32_t c = sh[b];
    if (c) atomicAdd(&g[b], c);
  }
}

// state[head][0] = threshold bin, [1] = tokens in bins above it, [2] = tokens still needed from it,
// [4] = candidates appended by the filter
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
  if (want == 0) {                                            // nothing to select: no bin is above or equal
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
  if (tid == FIN_THREADS - 1 && above + local < want) {       // fewer eligible tokens than wanted: take them all
    atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
    state[head * 8 + 0] = 0; state[head * 8 + 1] = above + local - c[3]; state[head * 8 + 2] = c[3];
  }
}

__global__ void __launch_bounds__(FILT_THREADS)
topk_filter_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   uint32_t* __restrict__ state, int32_t* __restrict__ cand, uint32_t* __restrict__ bitmap,
                   long long bitmap_words) {
  const int head = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t bstar = state[head * 8 + 0];
  const float* row = scores + (size_t)head * (size_t)score_stride;
  int32_t* cand_h = cand + (size_t)head * (size_t)n;
  uint32_t* bm = bitmap + (size_t)head * (size_t)bitmap_words;
  const long long wbase = (long long)blockIdx.x * FILT_TILE + (long long)warp * FILT_WARP_TOKENS;
  if (wbase >= n) return;
  uint32_t my_word = 0u;                                      // lane i keeps the ballot of iteration i
#pragma unroll 8
  for (int it = 0; it < 32; ++it) {
    const long long t = wbase + it * 32 + lane;
    const bool elig = t < n && t >= F.sink_end && t < F.local_begin;
    const float s = (t < n) ? __ldg(row + t) : 0.0f;
    const uint32_t bin = ordered_key(s) >> 20;
    const bool is_cand = elig && bin == bstar;
    const unsigned mw = __ballot_sync(0xffffffffu, elig && bin > bstar);
    const unsigned mc = __ballot_sync(0xffffffffu, is_cand);
    if (lane == it) my_word = mw;
    if (mc) {
      uint32_t pos = 0;
      const int leader = __ffs(mc) - 1;
      if (lane == leader) pos = atomicAdd(&state[head * 8 + 4], (uint32_t)__popc(mc));
      pos = __shfl_sync(0xffffffffu, pos, leader);
      if (is_cand) cand_h[pos + __popc(mc & ((1u << lane) - 1u))] = (int32_t)t;
    }
  }
  bm[wbase / 32 + lane] = my_word;                            // 32 consecutive words, one coalesced store
}

// low 52 bits of (key << 32 | ~index); the 12 leading key bits are the same for every candidate
__device__ __forceinline__ uint64_t composite52(const float* row, int32_t i) {
  return ((((uint64_t)ordered_key(row[i])) << 32) | (uint32_t)(~(uint32_t)i)) & ((1ull << 52) - 1ull);
}

__global__ void __launch_bounds__(FIN_THREADS)
topk_finish_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   const uint32_t* __restrict__ state, const int32_t* __restrict__ cand,
                   uint32_t* __restrict__ bitmap, long long bitmap_words, int k, int32_t* __restrict__ idx_out,
                   uint32_t* __restrict__ dev_status) {
  __shared__ uint64_t s_comp[FIN_CACHE];
  __shared__ uint32_t s_hist[256];
  __shared__ uint32_t s_warp[32];
  __shared__ uint64_t s_prefix;                               // decided leading bits of the threshold composite
  __shared__ uint32_t s_need, s_digit, s_bucket;
  const int head = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const int32_t* cand_h = cand + (size_t)head * (size_t)n;
  uint32_t* bm = bitmap + (size_t)head * (size_t)bitmap_words;
  const uint32_t m = state[head * 8 + 4];
  const uint32_t need0 = min(state[head * 8 + 2], m);
  const bool cached = m <= FIN_CACHE;
  if (cached)
    for (uint32_t c = tid; c < m; c += FIN_THREADS) s_comp[c] = composite52(row, cand_h[c]);

  // ---- radix select of the need0 largest composites among the m candidates; digits are taken from bit 52
  //      downwards (4 bits first, then 8 at a time) until the chosen bucket is taken whole.
  uint64_t thr = 0;                                           // chosen candidates: composite >= thr
  if (need0 > 0 && need0 < m) {
    if (tid == 0) { s_prefix = 0; s_need = need0; }
    int hi = 52;
    while (hi > 0) {
      const int bits = (hi % 8) ? (hi % 8) : 8;
      const int lo = hi - bits;
      if (tid < 256) s_hist[tid] = 0u;
      __syncthreads();
      const uint64_t prefix = s_prefix;
      for (uint32_t c = tid; c < m; c += FIN_THREADS) {
        const uint64_t comp = cached ? s_comp[c] : composite52(row, cand_h[c]);
        if ((comp >> hi) == (prefix >> hi)) atomicAdd(&s_hist[(uint32_t)(comp >> lo) & ((1u << bits) - 1u)], 1u);
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
            if (run < need && run + cnt[x] >= need) {
              s_digit = 255 - (8 * tid + x);
              s_need = need - run;                            // still needed from inside the chosen digit
              s_bucket = cnt[x];
            }
            run += cnt[x];
          }
        }
      }
      __syncthreads();
      if (tid == 0) s_prefix |= (uint64_t)s_digit << lo;
      const bool whole = s_need == s_bucket;                  // the chosen bucket is taken entirely: done
      __syncthreads();
      hi = lo;
      if (whole) break;
    }
    thr = s_prefix;                                           // undecided low bits are zero
  }
  if (need0 > 0) {
    for (uint32_t c = tid; c < m; c += FIN_THREADS) {
      const int32_t i = cand_h[c];
      const uint64_t comp = cached ? s_comp[c] : composite52(row, i);
      if (need0 >= m || comp >= thr) atomicOr(&bm[i >> 5], 1u << (i & 31));
    }
  }
  // ---- forced sink / local tokens
  const long long n_forced = F.sink_end + (n - F.local_begin);
  for (long long e = tid; e < n_forced; e += FIN_THREADS) {
    const long long i = (e < F.sink_end) ? e : (F.local_begin + (e - F.sink_end));
    atomicOr(&bm[i >> 5], 1u << (i & 31));
  }
  __syncthreads();

  // ---- ascending emission: thread t owns a contiguous run of bitmap words
  const long long words = (n + 31) / 32;
  const long long per = (words + FIN_THREADS - 1) / FIN_THREADS;
  const long long w0 = min((long long)tid * per, words), w1 = min(w0 + per, words);
  uint32_t cnt = 0;
  for (long long w = w0; w < w1; ++w) cnt += __popc(bm[w]);
  uint32_t incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const uint32_t w = s_warp[lane];
    uint32_t wi = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
      if (lane >= o) wi += y;
    }
    s_warp[lane] = wi - w;
    if (lane == 31 && wi != (uint32_t)k) atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
  }
  __syncthreads();
  uint32_t pos = s_warp[warp] + incl - cnt;
  int32_t* out = idx_out + (size_t)head * k;
  for (long long w = w0; w < w1; ++w) {
    uint32_t bitsw = bm[w];
    while (bitsw) {
      const int b = __ffs(bitsw) - 1;
      if (pos < (uint32_t)k) out[pos] = (int32_t)(w * 32 + b);
      ++pos;
      bitsw &= bitsw - 1;
    }
  }
  if (tid == FIN_THREADS - 1)                                 // short selection (non-finite scores): pad with the last token
    for (uint32_t e = pos; e < (uint32_t)k; ++e) out[e] = (int32_t)(n - 1);
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
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.bitmap - (char*)S.hist, st));
  dim3 hgrid((unsigned)((n + HIST_TILE - 1) / HIST_TILE), (unsigned)Hq);
  topk_hist_kernel<<<hgrid, HIST_THREADS, 0, st>>>(scores, n, L->score_stride, F, S.hist);
  topk_find_bin_kernel<<<Hq, FIN_THREADS, 0, st>>>(S.hist, S.state, want, ctx->dev_status);
  dim3 fgrid((unsigned)((n + FILT_TILE - 1) / FILT_TILE), (unsigned)Hq);
  topk_filter_kernel<<<fgrid, FILT_THREADS, 0, st>>>(scores, n, L->score_stride, F, S.state, S.cand, S.bitmap,
                                                     S.bitmap_words);
  topk_finish_kernel<<<Hq, FIN_THREADS, 0, st>>>(scores, n, L->score_stride, F, S.state, S.cand, S.bitmap,
                                                 S.bitmap_words, k, idx, ctx->dev_status);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
