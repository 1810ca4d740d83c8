// fathom_topk: per-query-head top-k over n scores with deterministic ties (Sec. 2 "Top-k decoding").
//
// Bucket select on the order-preserving integer image of the fp32 score (-0 folded onto +0):
//   1. histogram of the 12 leading key bits over all eligible tokens (one read of the scores); the CTA that
//      finishes a head's histogram last (ticket counter) finds
//   2. the threshold bin b* whose suffix count first reaches the number wanted;
//   3. filter (second read): a lane owns four consecutive tokens (one 16-byte load) and compares them with
//      the two fp32 edges of bin b*; the warp ballots of "above b*" ARE the words of a selection bitmap
//      (word c of a 128-token group holds tokens 4 l + c at bit l), written without atomics; tokens inside
//      bin b* are candidates, appended with warp-aggregated atomics (ballot + popc), order irrelevant;
//   4. per head, a radix select over the candidates on the 64-bit composite (key << 32 | ~index), which
//      makes every element distinct and encodes "ties go to the lower token index"; the chosen
//      candidates and the forced sink/local tokens are OR-ed into the bitmap and added to the per-tile
//      counts the filter left behind, whose prefix sum gives every tile its place in the output;
//   5. one small CTA per 8192-token tile emits its indices in ascending order (popcount prefix in the tile).
// The selected set is unique, so neither the append order nor atomics can show in the output.
#include "fathom_common.cuh"

namespace {

constexpr int HIST_THREADS = 256;
constexpr int HIST_TILE = 32768;                             // most scores per CTA of the histogram pass
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

__device__ void find_threshold_bin(const uint32_t* __restrict__ h, uint32_t* __restrict__ st, uint32_t want,
                                   uint32_t* __restrict__ dev_status, uint32_t* s_warp);

__global__ void __launch_bounds__(HIST_THREADS)
topk_hist_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                 uint32_t* __restrict__ hist, uint32_t* __restrict__ state, uint32_t want,
                 uint32_t* __restrict__ dev_status, int tile) {
  __shared__ uint32_t sh[FATHOM_TOPK_BINS];
  __shared__ bool s_last;
  const int head = blockIdx.y;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += HIST_THREADS) sh[b] = 0u;
  __syncthreads();
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const long long base = (long long)blockIdx.x * tile;         // tile: scores per CTA, a multiple of 1024
  const long long end = min(base + tile, n);
  // score_stride is a multiple of 4, so a float4 stays inside the row even when it straddles n
  if (base >= F.sink_end && base + tile <= F.local_begin) {   // whole tile eligible: no per-token test
    const float4* r4 = reinterpret_cast<const float4*>(row + base);
#pragma unroll 8
    for (int v = threadIdx.x; v < tile / 4; v += HIST_THREADS) {
      const float4 x = __ldg(r4 + v);
      atomicAdd(&sh[ordered_key(x.x) >> 20], 1u);
      atomicAdd(&sh[ordered_key(x.y) >> 20], 1u);
      atomicAdd(&sh[ordered_key(x.z) >> 20], 1u);
      atomicAdd(&sh[ordered_key(x.w) >> 20], 1u);
    }
  } else {
    for (long long i = base + (long long)threadIdx.x * 4; i < end; i += HIST_THREADS * 4) {
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
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += HIST_THREADS) {
    const uint32_t c = sh[b];
    if (c) atomicAdd(&g[b], c);
  }
  // the CTA that draws the head's last ticket sees the complete histogram and finds the threshold bin
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_last = atomicAdd(&state[head * 8 + 5], 1u) == gridDim.x - 1;
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  find_threshold_bin(g, state + head * 8, want, dev_status, sh);
}

// state[head][0] = threshold bin, [1] = tokens in bins above it, [2] = tokens still needed from it,
// [4] = candidates appended by the filter, [5] = ticket counter of the histogram CTAs.
// Run by the HIST_THREADS threads of the CTA that completed the head's histogram: thread t owns bins
// 4095 - 16 t .. 4080 - 16 t (descending), so a block prefix over threads is a suffix count over bins.
__device__ void find_threshold_bin(const uint32_t* __restrict__ h, uint32_t* __restrict__ st, uint32_t want,
                                   uint32_t* __restrict__ dev_status, uint32_t* s_warp) {
  constexpr int BPT = FATHOM_TOPK_BINS / HIST_THREADS;        // 16 bins per thread
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (want == 0) {                                            // nothing to select: no bin is above or equal
    if (tid == 0) { st[0] = FATHOM_TOPK_BINS; st[1] = 0; st[2] = 0; }
    return;
  }
  uint32_t c[BPT], local = 0;
#pragma unroll
  for (int x = 0; x < BPT; ++x) { c[x] = __ldcg(h + (FATHOM_TOPK_BINS - 1 - (BPT * tid + x))); local += c[x]; }
  uint32_t incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  uint32_t above = incl - local;
  for (int w = 0; w < warp; ++w) above += s_warp[w];          // 8 warps: a short serial carry
  if (above < want && above + local >= want) {
    uint32_t run = above;
#pragma unroll
    for (int x = 0; x < BPT; ++x) {
      if (run < want && run + c[x] >= want) {
        st[0] = (uint32_t)(FATHOM_TOPK_BINS - 1 - (BPT * tid + x));
        st[1] = run;
        st[2] = want - run;
      }
      run += c[x];
    }
  }
  if (tid == HIST_THREADS - 1 && above + local < want) {      // fewer eligible tokens than wanted: take them all
    atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
    st[0] = 0; st[1] = above + local - c[BPT - 1]; st[2] = c[BPT - 1];
  }
}

// fp32 value whose ordered key is `key` (the inverse of ordered_key for non-NaN patterns)
__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// Bitmap layout: word (t / 128) * 4 + (t % 4), bit (t % 128) / 4.
__device__ __forceinline__ long long bitmap_word(long long t) { return (t >> 7) * 4 + (t & 3); }
__device__ __forceinline__ uint32_t bitmap_bit(long long t) { return 1u << ((t & 127) >> 2); }

__global__ void __launch_bounds__(FILT_THREADS)
topk_filter_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   uint32_t* __restrict__ state, int32_t* __restrict__ cand, uint32_t* __restrict__ bitmap,
                   long long bitmap_words, uint32_t* __restrict__ tile_count) {
  __shared__ uint16_t s_list[FILT_TILE];                      // candidates of this tile, as offsets from its first token
  __shared__ uint32_t s_count, s_base, s_sel;
  const int head = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (threadIdx.x == 0) { s_count = 0u; s_sel = 0u; }
  __syncthreads();
  const uint32_t bstar = state[head * 8 + 0];
  // bin b* is [lo, hi) in fp32 order; for finite scores "key >> 20 > b*" <=> s >= hi and "== b*" <=> lo <= s < hi.
  // A bin edge that is not a number (beyond +-inf) compares false with everything, which is what is wanted.
  const float lo = (bstar < FATHOM_TOPK_BINS) ? key_to_float(bstar << 20) : __uint_as_float(0x7fc00000u);
  const float hi = (bstar + 1 < FATHOM_TOPK_BINS) ? key_to_float((bstar + 1) << 20) : __uint_as_float(0x7fc00000u);
  const bool hi_open = !(hi == hi);                           // no bin above b*: every s >= lo is a candidate
  const float* row = scores + (size_t)head * (size_t)score_stride;
  int32_t* cand_h = cand + (size_t)head * (size_t)n;
  uint32_t* bm = bitmap + (size_t)head * (size_t)bitmap_words;
  const long long tile0 = (long long)blockIdx.x * FILT_TILE;
  const long long wbase = tile0 + (long long)warp * FILT_WARP_TOKENS;
  const bool all_elig = wbase >= F.sink_end && wbase + FILT_WARP_TOKENS <= F.local_begin && wbase + FILT_WARP_TOKENS <= n;
  float4 x[FILT_WARP_TOKENS / 128];
#pragma unroll
  for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
    const long long t0 = wbase + it * 128 + lane * 4;
    x[it] = (t0 < n) ? __ldg(reinterpret_cast<const float4*>(row + t0)) : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  uint32_t my_word = 0u;                                      // lane w keeps word w of the warp's 32 bitmap words
  if (all_elig) {
#pragma unroll
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
      const float e[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
      const float mx = fmaxf(fmaxf(e[0], e[1]), fmaxf(e[2], e[3]));
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const unsigned mw = __ballot_sync(0xffffffffu, e[c] >= hi);
        if (lane == it * 4 + c) my_word = mw;
      }
      // candidates are rare (a few per thousand tokens): append them one by one to the tile's list
      if (mx >= lo) {                                          // divergent on purpose: only lanes that hold one
        const long long t0 = wbase + it * 128 + lane * 4;
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (e[c] >= lo && (hi_open || e[c] < hi)) s_list[atomicAdd(&s_count, 1u)] = (uint16_t)(t0 + c - tile0);
      }
    }
  } else {
#pragma unroll 1
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
      const long long t0 = wbase + it * 128 + lane * 4;
      const float e[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const long long t = t0 + c;
        const bool elig = t < n && t >= F.sink_end && t < F.local_begin;
        const bool is_cand = elig && e[c] >= lo && (hi_open || e[c] < hi);
        const unsigned mw = __ballot_sync(0xffffffffu, elig && e[c] >= hi);
        const unsigned mc = __ballot_sync(0xffffffffu, is_cand);
        if (lane == it * 4 + c) my_word = mw;
        if (mc) {
          uint32_t pos = 0;
          const int leader = __ffs(mc) - 1;
          if (lane == leader) pos = atomicAdd(&s_count, (uint32_t)__popc(mc));
          pos = __shfl_sync(0xffffffffu, pos, leader);
          if (is_cand) s_list[pos + __popc(mc & ((1u << lane) - 1u))] = (uint16_t)(t - tile0);
        }
      }
    }
  }
  if (wbase < n) bm[wbase / 32 + lane] = my_word;             // 32 consecutive words, one coalesced store
  {                                                           // tokens of this tile selected so far (bins above b*)
    uint32_t c = __popc(my_word);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
    if (lane == 0 && c) atomicAdd(&s_sel, c);
  }
  // one global atomic per tile reserves the slice of the head's candidate list
  __syncthreads();
  if (threadIdx.x == 0) tile_count[(size_t)head * gridDim.x + blockIdx.x] = s_sel;
  const uint32_t cnt = s_count;
  if (cnt == 0u) return;
  if (threadIdx.x == 0) s_base = atomicAdd(&state[head * 8 + 4], cnt);
  __syncthreads();
  const uint32_t base = s_base;
  for (uint32_t e = threadIdx.x; e < cnt; e += FILT_THREADS) cand_h[base + e] = (int32_t)(tile0 + s_list[e]);
}

// low 52 bits of (key << 32 | ~index); the 12 leading key bits are the same for every candidate
__device__ __forceinline__ uint64_t composite52(const float* row, int32_t i) {
  return ((((uint64_t)ordered_key(row[i])) << 32) | (uint32_t)(~(uint32_t)i)) & ((1ull << 52) - 1ull);
}

// Exclusive prefix over the block of one value per thread (warp shuffles + one shared array of 32 warp totals).
// Returns the exclusive prefix; *total receives the block sum.  Two __syncthreads.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* s_warp, uint32_t* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
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
    if (lane == 31) s_warp[32] = wi;
  }
  __syncthreads();
  *total = s_warp[32];
  return s_warp[warp] + incl - v;
}

// FUSED = false: candidates are the tokens of the threshold bin (their 12 leading key bits agree), scores are read
//                 from the dense score rows, the number needed comes from the histogram state.
// FUSED = true : candidates are (score, token) pairs collected by the filtering scan; `want_fused` of them are needed
//                 and the whole 64-bit composite takes part in the select.
template <bool FUSED>
__global__ void __launch_bounds__(FIN_THREADS)
topk_select_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   const uint32_t* __restrict__ state, const int32_t* __restrict__ cand,
                   uint32_t* __restrict__ bitmap, long long bitmap_words, int k, int32_t* __restrict__ idx_out,
                   uint32_t* __restrict__ dev_status, uint32_t* __restrict__ tile_count, int ntiles,
                   const uint32_t* __restrict__ cand_count, long long cand_capacity, uint32_t want_fused) {
  constexpr int DIGIT_BITS = 11, DIGITS = 1 << DIGIT_BITS;    // radix of the candidate select
  constexpr int DPT = DIGITS / FIN_THREADS;                    // digits per thread in the suffix scan
  __shared__ uint64_t s_comp[FIN_CACHE];
  __shared__ uint32_t s_hist[DIGITS];
  __shared__ uint32_t s_warp[33];
  __shared__ uint64_t s_prefix;                               // decided leading bits of the threshold composite
  __shared__ uint32_t s_need, s_bucket;
  const int head = blockIdx.x, tid = threadIdx.x;
  // dense: scores row of the head, candidate tokens [n];  fused: candidate scores and tokens [cand_capacity]
  const float* row = scores + (size_t)head * (size_t)(FUSED ? cand_capacity : score_stride);
  const int32_t* cand_h = cand + (size_t)head * (size_t)(FUSED ? cand_capacity : n);
  uint32_t* bm = bitmap + (size_t)head * (size_t)bitmap_words;
  uint32_t* tc = tile_count + (size_t)head * ntiles;
  const uint32_t m = FUSED ? (uint32_t)min((long long)cand_count[head], cand_capacity) : state[head * 8 + 4];
  const uint32_t need0 = min(FUSED ? want_fused : state[head * 8 + 2], m);
  constexpr int TOP = FUSED ? 64 : 52;                        // undecided bits of the composite
  auto composite = [&](uint32_t c) -> uint64_t {
    if (FUSED) return (((uint64_t)ordered_key(row[c])) << 32) | (uint32_t)(~(uint32_t)cand_h[c]);
    return composite52(row, cand_h[c]);
  };
  // The working set is either all m candidates in global memory or a subset kept in shared memory: everything when
  // m fits, otherwise the bucket of the first digit once it fits (what ranks above that bucket is marked at once).
  __shared__ uint32_t s_ncache;
  bool cached = m <= FIN_CACHE;
  uint32_t mc = m;                                            // size of the working set
  auto mark = [&](uint64_t comp) {                            // the token sits in the low 32 bits of every composite
    const int32_t i = (int32_t)~(uint32_t)comp;
    atomicOr(&bm[bitmap_word(i)], bitmap_bit(i));
    atomicAdd(&tc[i / FILT_TILE], 1u);
  };
  if (cached)
    for (uint32_t c = tid; c < m; c += FIN_THREADS) s_comp[c] = composite(c);

  // ---- radix select of the need0 largest composites among the m candidates: 11-bit digits from the top
  //      undecided bit downwards (the last digit is shorter) until the chosen bucket is taken whole.
  uint64_t thr = 0;                                           // chosen candidates: composite >= thr
  if (need0 > 0 && need0 < m) {
    if (tid == 0) { s_prefix = 0; s_need = need0; s_ncache = 0u; }
    int hi = TOP;
    while (hi > 0) {
      const int bits = min(DIGIT_BITS, hi);
      const int lo = hi - bits;
      for (int d = tid; d < DIGITS; d += FIN_THREADS) s_hist[d] = 0u;
      __syncthreads();
      const uint64_t prefix = s_prefix;
      const uint32_t need = s_need;
      // batches of 8 elements per thread: all loads of a batch are in flight together (one CTA serves a head, so
      // a load per loop iteration would leave the pass latency-bound)
      for (uint32_t c0 = 0; c0 < mc; c0 += FIN_THREADS * 8) {
        uint64_t comp[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t c = c0 + u * FIN_THREADS + tid;
          comp[u] = c < mc ? (cached ? s_comp[c] : composite(c)) : 0ull;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const uint32_t c = c0 + u * FIN_THREADS + tid;
          if (c < mc && (hi >= 64 || (comp[u] >> hi) == (prefix >> hi)))
            atomicAdd(&s_hist[(uint32_t)(comp[u] >> lo) & ((1u << bits) - 1u)], 1u);
        }
      }
      __syncthreads();
      // thread t owns digits DIGITS-1-DPT*t .. (descending): the block prefix is a suffix count
      uint32_t cnt[DPT], local = 0;
#pragma unroll
      for (int x = 0; x < DPT; ++x) { cnt[x] = s_hist[DIGITS - 1 - (DPT * tid + x)]; local += cnt[x]; }
      uint32_t total;
      uint32_t run = block_exclusive_scan(local, s_warp, &total);
      if (run < need && run + local >= need) {
#pragma unroll
        for (int x = 0; x < DPT; ++x) {
          if (run < need && run + cnt[x] >= need) {
            s_prefix = prefix | ((uint64_t)(DIGITS - 1 - (DPT * tid + x)) << lo);
            s_need = need - run;                              // still needed from inside the chosen digit
            s_bucket = cnt[x];
          }
          run += cnt[x];
        }
      }
      __syncthreads();
      hi = lo;
      if (s_need == s_bucket) break;                          // the chosen bucket is taken entirely: done
      if (!cached && s_bucket <= FIN_CACHE) {
        // the undecided bucket fits in shared memory: pull it in, mark what ranks above it, go on from there
        const uint64_t pfx = s_prefix;
        for (uint32_t c0 = 0; c0 < mc; c0 += FIN_THREADS * 8) {
          uint64_t comp[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t c = c0 + u * FIN_THREADS + tid;
            comp[u] = c < mc ? composite(c) : 0ull;
          }
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            const uint32_t c = c0 + u * FIN_THREADS + tid;
            const uint64_t top = hi >= 64 ? 0ull : (comp[u] >> hi), ptop = hi >= 64 ? 0ull : (pfx >> hi);
            if (c < mc && top > ptop) mark(comp[u]);
            const bool keep = c < mc && top == ptop;
            const unsigned km = __ballot_sync(0xffffffffu, keep);               // warp-aggregated append
            if (km) {
              uint32_t pos = 0;
              const int leader = __ffs(km) - 1;
              if ((tid & 31) == leader) pos = atomicAdd(&s_ncache, (uint32_t)__popc(km));
              pos = __shfl_sync(0xffffffffu, pos, leader);
              if (keep) s_comp[pos + __popc(km & ((1u << (tid & 31)) - 1u))] = comp[u];
            }
          }
        }
        __syncthreads();
        cached = true;
        mc = s_ncache;
      }
    }
    thr = s_prefix;                                           // undecided low bits are zero
  }
  if (need0 > 0) {
    for (uint32_t c = tid; c < mc; c += FIN_THREADS) {
      const uint64_t comp = cached ? s_comp[c] : composite(c);
      if (need0 >= m || comp >= thr) mark(comp);
    }
  }
  // ---- forced sink / local tokens
  const long long n_forced = F.sink_end + (n - F.local_begin);
  for (long long e = tid; e < n_forced; e += FIN_THREADS) {
    const long long i = (e < F.sink_end) ? e : (F.local_begin + (e - F.sink_end));
    atomicOr(&bm[bitmap_word(i)], bitmap_bit(i));
    atomicAdd(&tc[i / FILT_TILE], 1u);
  }
  __threadfence();
  __syncthreads();

  // ---- every tile's place in the output: exclusive prefix of the tile counts, in place
  uint32_t base = 0;
  for (int t0 = 0; t0 < ntiles; t0 += FIN_THREADS) {
    const int t = t0 + tid;
    const uint32_t c = (t < ntiles) ? __ldcg(tc + t) : 0u;
    uint32_t total;
    const uint32_t ex = block_exclusive_scan(c, s_warp, &total);
    if (t < ntiles) tc[t] = base + ex;
    base += total;
    __syncthreads();
  }
  if (base != (uint32_t)k && tid == 0) {                      // short selection (non-finite scores)
    atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
    int32_t* out = idx_out + (size_t)head * k;
    for (uint32_t e = base; e < (uint32_t)k; ++e) out[e] = (int32_t)(n - 1);   // pad with the last token
  }
}

// One CTA per (tile of FILT_TILE tokens, head): thread = group of 128 tokens (4 bitmap words, one 16-byte load).
__global__ void __launch_bounds__(FILT_TILE / 128)
topk_emit_kernel(const uint32_t* __restrict__ bitmap, long long bitmap_words, const uint32_t* __restrict__ tile_offset,
                 long long n, int k, int32_t* __restrict__ idx_out) {
  constexpr int EMIT_THREADS = FILT_TILE / 128;               // 64
  __shared__ uint32_t s_w[EMIT_THREADS / 32];
  const int head = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long g = (long long)blockIdx.x * EMIT_THREADS + tid;
  const long long groups = (n + 127) / 128;
  const uint4* bm4 = reinterpret_cast<const uint4*>(bitmap + (size_t)head * (size_t)bitmap_words);
  const uint4 w = (g < groups) ? __ldcg(bm4 + g) : make_uint4(0u, 0u, 0u, 0u);
  const uint32_t c = __popc(w.x) + __popc(w.y) + __popc(w.z) + __popc(w.w);
  uint32_t incl = c;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_w[warp] = incl;
  __syncthreads();
  uint32_t pos = tile_offset[(size_t)head * gridDim.x + blockIdx.x] + incl - c;
  for (int x = 0; x < warp; ++x) pos += s_w[x];
  int32_t* out = idx_out + (size_t)head * k;
  uint32_t any = w.x | w.y | w.z | w.w;
  while (any) {
    const int l = __ffs(any) - 1;
    any &= any - 1;
    const int32_t t = (int32_t)(g * 128 + 4 * l);
    if ((w.x >> l) & 1u) { if (pos < (uint32_t)k) out[pos] = t; ++pos; }
    if ((w.y >> l) & 1u) { if (pos < (uint32_t)k) out[pos] = t + 1; ++pos; }
    if ((w.z >> l) & 1u) { if (pos < (uint32_t)k) out[pos] = t + 2; ++pos; }
    if ((w.w >> l) & 1u) { if (pos < (uint32_t)k) out[pos] = t + 3; ++pos; }
  }
}

}  // namespace

// Scores per histogram CTA: large tiles amortise the 4096-bin flush, but short rows still need a few hundred CTAs.
static int hist_tile_for(long long n, int Hq) {
  long long tile = HIST_TILE;
  while (tile > 4096 && ((n + tile - 1) / tile) * Hq < 600) tile /= 2;
  return (int)tile;
}

// Dense selection over score rows (the four launches of fathom_topk).
static int run_dense_topk(fathom_ctx* ctx, const float* scores, long long n, long long score_stride, int Hq, int k,
                          Forced F, uint32_t want, const fathom_topk_scratch& S, int32_t* idx, cudaStream_t st) {
  // histograms, per-head state and candidate counters are contiguous at the start of the arena
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.bitmap - (char*)S.hist, st));
  const int htile = hist_tile_for(n, Hq);
  dim3 hgrid((unsigned)((n + htile - 1) / htile), (unsigned)Hq);
  topk_hist_kernel<<<hgrid, HIST_THREADS, 0, st>>>(scores, n, score_stride, F, S.hist, S.state, want, ctx->dev_status, htile);
  const int ntiles = (int)((n + FILT_TILE - 1) / FILT_TILE);
  dim3 fgrid((unsigned)ntiles, (unsigned)Hq);
  topk_filter_kernel<<<fgrid, FILT_THREADS, 0, st>>>(scores, n, score_stride, F, S.state, S.cand, S.bitmap, S.bitmap_words,
                                                     S.tile_count);
  topk_select_kernel<false><<<Hq, FIN_THREADS, 0, st>>>(scores, n, score_stride, F, S.state, S.cand, S.bitmap, S.bitmap_words,
                                                        k, idx, ctx->dev_status, S.tile_count, ntiles, nullptr, 0, 0u);
  topk_emit_kernel<<<fgrid, FILT_TILE / 128, 0, st>>>(S.bitmap, S.bitmap_words, S.tile_count, n, k, idx);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

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
  fathom_topk_scratch S = fathom_carve_topk(ctx->scratch, L->n_q_heads, n, k);
  if (S.bytes > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  return run_dense_topk(ctx, scores, n, L->score_stride, L->n_q_heads, k, F, (uint32_t)(k - n_forced), S, idx,
                        static_cast<cudaStream_t>(stream));
}

// Tile step of the sample scan for (n, k): every 16th scan tile when that sample still holds at least 2 k tokens,
// otherwise 1 (the "sample" is then the whole score array and the dense selection runs on it).
int fathom_fused_tile_step(long long n, int k) {
  const long long tile = fathom_scan_tile_tokens();
  const long long ntiles = (n + tile - 1) / tile;
  const long long sampled = (ntiles + 15) / 16;                       // tiles 0, 16, 32, ...
  const long long last_start = (sampled - 1) * 16 * tile;             // first token of the last sampled tile (< n)
  const long long valid = (sampled - 1) * tile + ((n - last_start) < tile ? (n - last_start) : tile);
  return (ntiles >= 16 && valid >= 2LL * k) ? 16 : 1;
}

extern "C" int fathom_scan_topk(fathom_ctx* ctx, const fathom_layout* L, const uint64_t* planes, const uint16_t* scales,
                                const float* q, const uint8_t* depth, int heads_per_plan, int k, int n_sink, int n_local,
                                int32_t* idx, void* stream) {
  if (!ctx || !planes || !scales || !q || !depth || !idx) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  const int Hq = L->n_q_heads, G = Hq / L->n_kv_heads;
  if (heads_per_plan < 1 || G % heads_per_plan != 0) return FATHOM_ERR_INVALID_ARG;
  if (heads_per_plan != 1 && heads_per_plan != 2 && heads_per_plan != 4 && heads_per_plan != 8) return FATHOM_ERR_UNSUPPORTED;
  if (k < 1 || k > L->n || k > FATHOM_MAX_K || n_sink < 0 || n_local < 0) return FATHOM_ERR_INVALID_ARG;
  if (!fathom_aligned16(planes) || !fathom_aligned16(scales)) return FATHOM_ERR_ALIGNMENT;
  const long long n = L->n;
  Forced F;
  F.sink_end = n_sink < n ? n_sink : n;
  F.local_begin = (n - n_local > F.sink_end) ? (n - n_local) : F.sink_end;
  const long long n_forced = F.sink_end + (n - F.local_begin);
  if (n_forced > k) return FATHOM_ERR_INVALID_ARG;
  fathom_topk_scratch S = fathom_carve_topk(ctx->scratch, Hq, n, k);
  if (S.bytes > ctx->scratch_bytes) return FATHOM_ERR_SCRATCH_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const uint32_t want = (uint32_t)(k - n_forced);
  const int step = fathom_fused_tile_step(n, k);
  const long long tile = fathom_scan_tile_tokens();
  const long long ntiles_scan = (n + tile - 1) / tile;

  // ---- sample: scores of every `step`-th scan tile, compact
  rc = fathom_launch_scan_sample(L, planes, scales, q, depth, heads_per_plan, S.sample, S.sample_stride, step, st);
  if (rc != FATHOM_OK) return rc;
  if (step == 1)                                              // short sequence: the sample is the whole score array
    return run_dense_topk(ctx, S.sample, n, S.sample_stride, Hq, k, F, want, S, idx, st);

  // ---- threshold: the bin in which the sample's k-th largest score lies.  At least k tokens of the sample, hence
  //      at least k - n_forced eligible tokens of the sequence, reach its lower edge: no winner can lie below it.
  const long long sampled = (ntiles_scan + step - 1) / step;
  const long long last_start = (sampled - 1) * step * tile;
  const long long n_sample = (sampled - 1) * tile + ((n - last_start) < tile ? (n - last_start) : tile);
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.bitmap - (char*)S.hist, st));
  Forced none;
  none.sink_end = 0;
  none.local_begin = n_sample;
  const int htile = hist_tile_for(n_sample, Hq);
  dim3 hgrid((unsigned)((n_sample + htile - 1) / htile), (unsigned)Hq);
  topk_hist_kernel<<<hgrid, HIST_THREADS, 0, st>>>(S.sample, n_sample, S.sample_stride, none, S.hist, S.state, (uint32_t)k,
                                                   ctx->dev_status, htile);
  // ---- full scan that keeps only the tokens reaching their head's threshold
  const int ntiles = (int)((n + FILT_TILE - 1) / FILT_TILE);
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.bitmap, 0, (size_t)Hq * S.bitmap_words * 4, st));
  FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.tile_count, 0, (size_t)Hq * ntiles * 4, st));
  fathom_scan_fuse fz = {};
  fz.tile_step = 1;
  fz.state = S.state;
  fz.sink_end = F.sink_end;
  fz.local_begin = F.local_begin;
  fz.cand_score = S.cand_score;
  fz.cand_idx = S.cand;
  fz.cand_count = S.cand_count;
  fz.capacity = n;
  rc = fathom_launch_scan_filter(L, planes, scales, q, depth, heads_per_plan, fz, st);
  if (rc != FATHOM_OK) return rc;
  // ---- exact selection among the candidates, then ascending emission
  topk_select_kernel<true><<<Hq, FIN_THREADS, 0, st>>>(S.cand_score, n, 0, F, S.state, S.cand, S.bitmap, S.bitmap_words, k, idx,
                                                       ctx->dev_status, S.tile_count, ntiles, S.cand_count, n, want);
  dim3 fgrid((unsigned)ntiles, (unsigned)Hq);
  topk_emit_kernel<<<fgrid, FILT_TILE / 128, 0, st>>>(S.bitmap, S.bitmap_words, S.tile_count, n, k, idx);
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
