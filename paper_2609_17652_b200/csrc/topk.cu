// fathom_topk: per-query-head top-k over n scores with deterministic ties (Sec. 2 "Top-k decoding").
//
// Both paths select on the order-preserving integer image of the fp32 score (-0 folded onto +0), and both give the
// one set the definition fixes (ties to the lower token index), in ascending token order.
//
// Single pass (rows of 64K scores or more, at least 256 wanted): one read of the scores.
//   a. a cluster of four CTAs per head histograms every 16th 1024-score chunk (12 leading key bits, shared memory,
//      merged through distributed shared memory) and finds two bins:
//      the ESTIMATE, whose suffix count in the sample reaches the expected rank plus four standard deviations, and
//      the BOUND, whose suffix count reaches k in the sample alone and therefore in the whole row;
//   b. every CTA of the collection pass loads its 8192 scores before the sample kernel has finished (programmatic
//      dependent launch), marks its candidates (scores that reach the estimate's lower edge), gives each a place by a
//      prefix count over the CTA and ONE atomic on the head's counter, and appends the (score, token) pairs;
//   c. per head, one CTA selects among the list on the composite (key << 32 | ~index).  The short way (lists of up to
//      16384, sequences whose bitmap fits in shared memory): a fine histogram of the candidates' distance from the
//      threshold finds the bin of the wanted-th largest, the few members of that bin are ranked against one another,
//      the chosen tokens are set in a bitmap and read off it in ascending order with popcounts.  The general way: a
//      radix select over the list (11-bit digits; a chosen digit with few members is finished by ranking them), the
//      winners placed in ascending order by a counting sort over 4096 token ranges.  A head whose list came out
//      shorter than wanted (the estimate was too high) collects again itself above the bound bin, which cannot fall
//      short.
//
// Two passes (short rows, or FATHOM_TOPK_PATH=two_pass): bucket select.
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

#include <cooperative_groups.h>

#include <cmath>
#include <cstdlib>
#include <cstring>

namespace cg = cooperative_groups;

namespace {

constexpr int HIST_THREADS = 256;
constexpr int HIST_TILE = 32768;                             // most scores per CTA of the histogram pass
constexpr int FILT_THREADS = 256;
constexpr int FILT_WARP_TOKENS = 1024;                       // 32 ballots -> 32 bitmap words per warp
constexpr int FILT_TILE = (FILT_THREADS / 32) * FILT_WARP_TOKENS;   // 8192 tokens per CTA
constexpr int FIN_THREADS = 1024;
constexpr int FIN_CACHE = 8192;                              // candidate composites kept in shared memory: two-pass select (64 KB)
constexpr int FIN_CACHE_MAX = 16384;                         // ... direct select, when k leaves room (128 KB)

__device__ __forceinline__ uint32_t ordered_key(float f) {
  uint32_t u = __float_as_uint(f);
  if ((u << 1) == 0u) u = 0u;                                // -0 -> +0
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// fp32 value whose ordered key is `key` (the inverse of ordered_key for non-NaN patterns)
__device__ __forceinline__ float key_to_float(uint32_t key) {
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}
// Lower edge of a histogram bin as a score: the bins below -inf's (no finite score lies there) stand for "every score",
// a bin past the last for "none" (a comparison with NaN is false).
__device__ __forceinline__ float edge_of_bin(uint32_t bin) {
  return bin >= FATHOM_TOPK_BINS ? __uint_as_float(0x7fc00000u) : (bin <= 7u ? -INFINITY : key_to_float(bin << 20));
}

struct Forced { long long sink_end, local_begin; };          // eligible tokens: sink_end <= i < local_begin

using Gate = fathom_gate;

template <int THREADS, bool IN_GLOBAL>
__device__ void find_threshold_bin(const uint32_t* __restrict__ h, uint32_t* __restrict__ st, uint32_t want,
                                   uint32_t* __restrict__ dev_status, uint32_t* s_warp, uint32_t want_bound);

// A CTA histograms `reps` tiles of `tile` scores that start cta_stride tokens apart (cta_stride = tile, reps = 1 for a
// full pass; a multiple of the tile when only every m-th tile is histogrammed to estimate a threshold, in which case
// dev_status is NULL: a short sample is no error).
__global__ void __launch_bounds__(HIST_THREADS)
topk_hist_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                 uint32_t* __restrict__ hist, uint32_t* __restrict__ state, uint32_t want,
                 uint32_t* __restrict__ dev_status, int tile, long long cta_stride, int reps, uint32_t want_bound) {
  __shared__ uint32_t sh[FATHOM_TOPK_BINS];
  __shared__ bool s_last;
  const int head = blockIdx.y;
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += HIST_THREADS) sh[b] = 0u;
  __syncthreads();
  const float* row = scores + (size_t)head * (size_t)score_stride;
  // score_stride is a multiple of 4, so a float4 stays inside the row even when it straddles n
  const long long first = (long long)blockIdx.x * reps * cta_stride;
  if (reps > 1) {
    // sampled tiles (those that lie wholly inside the row), walked as one index space so that the loads of different
    // tiles are in flight together.  Forced tokens are not told apart here: the caller asks for a bound rank that
    // allows for all of them.
    const int per_tile = tile / 4, pt_shift = 31 - __clz(per_tile);   // tile is a power of two
#pragma unroll 8
    for (int v = threadIdx.x; v < reps * per_tile; v += HIST_THREADS) {
      const long long tb = first + (long long)(v >> pt_shift) * cta_stride;
      if (tb + tile <= n) {
        const float4 x = __ldg(reinterpret_cast<const float4*>(row + tb) + (v & (per_tile - 1)));
        atomicAdd(&sh[ordered_key(x.x) >> 20], 1u);
        atomicAdd(&sh[ordered_key(x.y) >> 20], 1u);
        atomicAdd(&sh[ordered_key(x.z) >> 20], 1u);
        atomicAdd(&sh[ordered_key(x.w) >> 20], 1u);
      }
    }
  } else {
    const long long base = first;
    const long long end = min(base + tile, n);
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
  find_threshold_bin<HIST_THREADS, true>(g, state + head * 8, want, dev_status, sh, want_bound);
}

// state[head][0] = threshold bin, [1] = tokens in bins above it, [2] = tokens still needed from it, [3] = bound bin
// of a sampled histogram, [4] = candidates appended by the filter, [5] = ticket counter of the histogram CTAs,
// [6] = the score a candidate of the first attempt must reach (fp32 bits): the lower edge of bin [0].
// Run by all THREADS threads of a CTA that sees the head's complete histogram h (in global memory: the CTA that
// finished it last; or in shared memory): thread t owns bins 4095 - BPT t .. (descending), so a block prefix over
// threads is a suffix count over bins.  s_warp: at least THREADS / 32 words of shared memory.
// want: rank whose bin goes to words 0..2.  want_bound (0 = none): rank whose bin alone goes to word 3 (histogram of
// a sample: the bin of the sample's want_bound-th largest score is reached by at least that many tokens of the row).
template <int THREADS, bool IN_GLOBAL>
__device__ void find_threshold_bin(const uint32_t* __restrict__ h, uint32_t* __restrict__ st, uint32_t want,
                                   uint32_t* __restrict__ dev_status, uint32_t* s_warp, uint32_t want_bound) {
  constexpr int BPT = FATHOM_TOPK_BINS / THREADS;             // bins per thread
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t c[BPT], local = 0;
#pragma unroll
  for (int x = 0; x < BPT; ++x) {                             // a histogram other CTAs added to is read past the L1
    const uint32_t* p = h + (FATHOM_TOPK_BINS - 1 - (BPT * tid + x));
    c[x] = IN_GLOBAL ? __ldcg(p) : *p;
    local += c[x];
  }
  uint32_t incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  uint32_t above = incl - local;
  {                                                           // + the totals of the warps before mine (lane l sums warp l's if l < warp)
    uint32_t carry = (lane < warp && lane < THREADS / 32) ? s_warp[lane] : 0u;
#pragma unroll
    for (int o = 16; o; o >>= 1) carry += __shfl_xor_sync(0xffffffffu, carry, o);
    above += carry;
  }
  auto search = [&](uint32_t rank, bool bound_slot) {
    if (rank == 0) {                                          // nothing to select: no bin is above or equal
      if (tid == 0) {
        if (bound_slot) st[3] = FATHOM_TOPK_BINS;
        else { st[0] = FATHOM_TOPK_BINS; st[1] = 0; st[2] = 0; st[6] = __float_as_uint(edge_of_bin(FATHOM_TOPK_BINS)); }
      }
      return;
    }
    if (above < rank && above + local >= rank) {
      uint32_t run = above;
#pragma unroll
      for (int x = 0; x < BPT; ++x) {
        if (run < rank && run + c[x] >= rank) {
          const uint32_t bin = (uint32_t)(FATHOM_TOPK_BINS - 1 - (BPT * tid + x));
          if (bound_slot) st[3] = bin;
          else { st[0] = bin; st[1] = run; st[2] = rank - run; st[6] = __float_as_uint(edge_of_bin(bin)); }
        }
        run += c[x];
      }
    }
    if (tid == THREADS - 1 && above + local < rank) {         // fewer tokens than wanted: take them all
      if (!bound_slot && dev_status) atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
      if (bound_slot) st[3] = 0;
      else { st[0] = 0; st[1] = above + local - c[BPT - 1]; st[2] = c[BPT - 1]; st[6] = __float_as_uint(edge_of_bin(0u)); }
    }
  };
  search(want, false);
  if (want_bound) search(want_bound, true);
}

// Histogram of a head's sample (every 16th whole chunk of 1024 scores) by a cluster of SAMPLE_CLUSTER CTAs: each
// histograms its share of the chunks in its own shared memory, the others add their non-empty bins to the first CTA's
// through distributed shared memory (atomics: a few hundred bins of 4096 hold anything), and the first CTA finds the
// estimated and the bound bin: no global histogram, no flush, no ticket.  For rows of up to a few million scores.
constexpr int SAMPLE_THREADS = 1024;
constexpr int SAMPLE_CLUSTER = 4;
__global__ void __cluster_dims__(SAMPLE_CLUSTER, 1, 1) __launch_bounds__(SAMPLE_THREADS)
topk_sample_kernel(const float* __restrict__ scores, long long sampled, long long chunk_stride, long long score_stride,
                   uint32_t* __restrict__ state, uint32_t want, uint32_t want_bound, uint32_t* __restrict__ cand_count,
                   uint32_t* __restrict__ cand_count2) {
  __shared__ uint32_t sh[FATHOM_TOPK_BINS];
  __shared__ uint32_t s_warp[SAMPLE_THREADS / 32];
  cg::cluster_group cluster = cg::this_cluster();
  const int head = blockIdx.x / SAMPLE_CLUSTER, part = (int)cluster.block_rank();
  FATHOM_PDL_WAIT();                                          // the scores come from the previous kernel (this one may be launched as its dependent)
  // the collection kernel may be launched as a programmatic dependent: let it start at once, it loads its scores while
  // this kernel runs and waits for this kernel's results only before it compares
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (part == 0 && threadIdx.x == 0) {                        // the collection that follows counts from zero
    cand_count[head] = 0u;
    if (cand_count2) cand_count2[head] = 0u;
  }
  for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += SAMPLE_THREADS) sh[b] = 0u;
  __syncthreads();
  auto cleared = cluster.barrier_arrive();                    // my histogram is clear (the first CTA's will be added to)
  const float* row = scores + (size_t)head * (size_t)score_stride;
  // `sampled` whole chunks of 1024 scores, chunk_stride scores apart (16384: every 16th chunk of a score row; 1024: a
  // compact array of sampled scores); CTA `part` of the cluster takes every SAMPLE_CLUSTER-th group of 1024 float4
#pragma unroll 4
  for (long long v = (long long)part * SAMPLE_THREADS + threadIdx.x; v < sampled * 256; v += SAMPLE_CLUSTER * SAMPLE_THREADS) {
    const float4 x = __ldg(reinterpret_cast<const float4*>(row + (v >> 8) * chunk_stride) + (v & 255));
    atomicAdd(&sh[ordered_key(x.x) >> 20], 1u);
    atomicAdd(&sh[ordered_key(x.y) >> 20], 1u);
    atomicAdd(&sh[ordered_key(x.z) >> 20], 1u);
    atomicAdd(&sh[ordered_key(x.w) >> 20], 1u);
  }
  __syncthreads();                                            // my histogram is complete
  cluster.barrier_wait(std::move(cleared));                   // (everyone arrived long ago: no wait in practice)
  if (part != 0) {                                            // my non-empty bins are added to the first CTA's: a few hundred of 4096
    uint32_t* first = cluster.map_shared_rank(sh, 0);
    for (int b = threadIdx.x; b < FATHOM_TOPK_BINS; b += SAMPLE_THREADS) {
      const uint32_t c = sh[b];
      if (c) atomicAdd(first + b, c);
    }
  }
  cluster.sync();                                             // the additions are complete and visible
  if (part != 0) return;
  find_threshold_bin<SAMPLE_THREADS, false>(sh, state + head * 8, want, nullptr, s_warp, want_bound);
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

// Collection pass of the single-pass top-k: every eligible token whose score reaches the head's estimated threshold
// (state word 6, from the histogram of every 16th chunk) is appended to the head's candidate list as a (score, token)
// pair.
__global__ void __launch_bounds__(FILT_THREADS, 5)
topk_collect_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                    const uint32_t* state, float* __restrict__ cand_score, int32_t* __restrict__ cand_idx,
                    uint32_t* __restrict__ cand_count, int ntiles) {
  __shared__ uint32_t s_warp_total[FILT_THREADS / 32];
  __shared__ uint32_t s_base;
  // one CTA per (head, tile): grid = (heads, tiles in y and z), tiles from the last to the first and all heads of a tile
  // together: the scan writes the heads' rows side by side from the first token to the last, so what it wrote last is
  // the likeliest to be in L2 still
  const int head = gridDim.x - 1 - blockIdx.x;
  const int tile = ntiles - 1 - (int)(blockIdx.z * gridDim.y + blockIdx.y);
  if (tile < 0) return;                                        // padding of the last z slice
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float* row = scores + (size_t)head * (size_t)score_stride;
  const long long tile0 = (long long)tile * FILT_TILE;
  const long long wbase = tile0 + (long long)warp * FILT_WARP_TOKENS;
  const bool all_elig = wbase >= F.sink_end && wbase + FILT_WARP_TOKENS <= F.local_begin && wbase + FILT_WARP_TOKENS <= n;
  float4 x[FILT_WARP_TOKENS / 128];
  if (wbase + FILT_WARP_TOKENS <= n) {                        // (uniform over the warp) no load needs a guard
    const float4* src = reinterpret_cast<const float4*>(row + wbase) + lane;
#pragma unroll
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) x[it] = __ldcs(src + it * 32);     // read once: first to be evicted
  } else {
#pragma unroll
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
      const long long t0 = wbase + it * 128 + lane * 4;
      x[it] = (t0 < n) ? __ldcs(reinterpret_cast<const float4*>(row + t0)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  // The scores were complete before the sample kernel started; its threshold and cleared counters are needed from
  // here on (a no-op unless this kernel was launched as a programmatic dependent of the sample kernel).
  FATHOM_PDL_WAIT();
  FATHOM_PDL_RELEASE();                                       // the selection that follows may become resident now
  const float lo = __uint_as_float(__ldcg(state + head * 8 + 6));   // the score a candidate must reach
  // ---- which of my 32 scores are candidates (bit 4 it + c), then a place for each: my candidates follow those of the
  //      lanes before me, the warp's those of the warps before it, the CTA's block comes from ONE atomic on the head's count
  uint32_t mine = 0;
  if (all_elig) {                                             // (uniform over the warp) nothing else to check
#pragma unroll
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
      mine |= (x[it].x >= lo ? 1u : 0u) << (4 * it);
      mine |= (x[it].y >= lo ? 1u : 0u) << (4 * it + 1);
      mine |= (x[it].z >= lo ? 1u : 0u) << (4 * it + 2);
      mine |= (x[it].w >= lo ? 1u : 0u) << (4 * it + 3);
    }
  } else {
#pragma unroll
    for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
      const float e[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        const long long t = wbase + it * 128 + lane * 4 + c;
        mine |= (e[c] >= lo && t < n && t >= F.sink_end && t < F.local_begin ? 1u : 0u) << (4 * it + c);
      }
    }
  }
  const uint32_t cnt = __popc(mine);
  uint32_t incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += y;
  }
  if (lane == 31) s_warp_total[warp] = incl;
  __syncthreads();
  uint32_t before = 0, total = 0;
#pragma unroll
  for (int w = 0; w < FILT_THREADS / 32; ++w) {
    const uint32_t c = s_warp_total[w];
    before += w < warp ? c : 0u;
    total += c;
  }
  if (total == 0u) return;                                    // (the same for every thread)
  if (threadIdx.x == 0) s_base = atomicAdd(&cand_count[head], total);
  __syncthreads();
  if (mine == 0u || (long long)s_base + total > n) return;    // (a list holds at most n: every token is appended once per call)
  uint32_t pos = s_base + before + incl - cnt;
  float* cs = cand_score + (size_t)head * (size_t)n;
  int32_t* ci = cand_idx + (size_t)head * (size_t)n;
#pragma unroll
  for (int it = 0; it < FILT_WARP_TOKENS / 128; ++it) {
    const float e[4] = {x[it].x, x[it].y, x[it].z, x[it].w};
    if ((mine >> (4 * it)) & 15u) {
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if ((mine >> (4 * it + c)) & 1u) {
          cs[pos] = e[c];
          ci[pos] = (int32_t)(wbase + it * 128 + lane * 4 + c);
          ++pos;
        }
    }
  }
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


// The short way of the direct select, for a head whose candidates had to reach a known score `lo`.  FAST_PARTS CTAs
// share a head without talking to one another: each loads all the candidates and finds the threshold itself, then
// emits the chosen tokens of its own quarter of the sequence.
// The candidates (at most 16 per thread, loaded once, kept in registers as bin and token) are counted in a fine
// histogram of the key's distance from lo's key (2048 bins of 2^13 keys: 16 bins of the 12-bit histogram lo came from;
// the last bin takes everything beyond).  Its suffix counts give the bin b that holds the wanted-th largest candidate;
// candidates in bins above b are chosen at once, the few dozen members of b are listed and ranked against one another
// on the composite (key << 32 | ~token).  A chosen token of the CTA's own quarter is set in a bitmap in shared memory,
// one before the quarter is counted; the quarter's tokens are then read off the bitmap in ascending order, each thread
// its own groups, at the place given by the count before the quarter plus the popcounts of the threads before it: one
// histogram pass over the candidates, no sort.  Everything needed from global memory is requested before anything is
// waited for.  Returns false, with nothing but the cleared bitmap and histogram touched, when it does not apply (the
// same for all CTAs of a head): the head has to collect again (too few candidates), more than 16 candidates per
// thread, or a bin b with more than SMALL members.  The head's first CTA then selects the general way.
// Shared memory: bitmap of 1024 U 16-byte groups (U per thread), one group skipped after every 8 so that the threads of
// a quarter warp, each reading its own U consecutive groups, hit different banks.
constexpr int FINE_BINS = 2048, FINE_SHIFT = 13;
__device__ __forceinline__ uint32_t fine_bin(float score, float lo) {
  const uint32_t key = ordered_key(score), base = ordered_key(lo);
  return min((key > base ? key - base : 0u) >> FINE_SHIFT, (uint32_t)(FINE_BINS - 1));
}
constexpr int FAST_PARTS = 4;                                 // CTAs per head
constexpr int FAST_MAXU = 4;                                  // 16-byte bitmap groups per thread
constexpr long long FAST_MAX_TOKENS = (1ll << 21) - 1;        // tokens are kept in 21 bits
// 16-byte groups (128 tokens) of a part, and per thread of it
__host__ __device__ inline long long fast_part_groups(long long n) { return ((n + 127) / 128 + FAST_PARTS - 1) / FAST_PARTS; }
__host__ __device__ inline long long fast_select_groups(long long n) { return (fast_part_groups(n) + FIN_THREADS - 1) / FIN_THREADS; }   // U
__host__ __device__ inline long long fast_select_bytes(long long n) {
  const long long G = fast_select_groups(n) * FIN_THREADS;
  return (G + (G >> 3)) * 16;
}
static_assert(FAST_MAX_TOKENS <= (long long)FAST_PARTS * FAST_MAXU * FIN_THREADS * 128, "the parts' bitmaps must cover every token");
constexpr int FAST_EPT = 8;                                   // candidates per thread and round of loads
// ROUNDS = 1: lists of up to 8192 candidates; 2: up to 16384 (a second round of loads once the length is known)
template <int SMALL, int ROUNDS>
__device__ __forceinline__ bool select_by_fine_histogram_rounds(
    const float* __restrict__ cs, const int32_t* __restrict__ ci, uint32_t m, const float (&sc0)[FAST_EPT], const int32_t (&ix0)[FAST_EPT],
    uint32_t want, float lo, long long n, int k, int part,
    Forced F, unsigned char* s_dyn, uint32_t* s_fine, uint32_t* s_warp, int32_t* __restrict__ out, uint32_t* __restrict__ dev_status) {
  constexpr int EPT = FAST_EPT;
  constexpr int FPT = FINE_BINS / FIN_THREADS;                 // fine bins per thread
  constexpr uint32_t TOKEN_BITS = 21, NONE = 0xffffffffu;      // a candidate in a register: fine bin << 21 | token
  static_assert(FAST_MAX_TOKENS <= (1ll << TOKEN_BITS) - 1, "tokens must fit beside the bin, NONE must be no token");
  static_assert(SMALL * 8 <= FINE_BINS * 4, "the members of the split bin are listed where the fine histogram was");
  __shared__ uint32_t s_bin, s_need_in, s_members, s_nsmall;
  uint64_t* s_small = reinterpret_cast<uint64_t*>(s_fine);     // (free once every thread has read its bins)
  const int tid = threadIdx.x;
  const uint32_t U = (uint32_t)fast_select_groups(n);
  const uint32_t first_token = (uint32_t)part * (uint32_t)fast_part_groups(n) * 128u;   // my part: [first_token, + part_tokens)
  const uint32_t part_tokens = (uint32_t)fast_part_groups(n) * 128u;
  uint32_t* s_bits = reinterpret_cast<uint32_t*>(s_dyn);
  const uint4* s_bits4 = reinterpret_cast<const uint4*>(s_dyn);
  auto group_at = [](uint32_t g) { return g + (g >> 3); };     // where group g of the bitmap sits
  uint32_t below = 0;                                         // chosen tokens before my part (my share of the count)
  auto choose = [&](uint32_t t) {                              // a chosen token: into the bitmap, counted, or not mine to emit
    const uint32_t r = t - first_token;
    if (t < first_token) ++below;
    else if (r < part_tokens) {
      const uint32_t w = r >> 5;
      atomicOr(&s_bits[(group_at(w >> 2) << 2) | (w & 3u)], 1u << (r & 31u));
    }
  };
  uint32_t cand[ROUNDS * EPT];
  if (tid == 0) { s_nsmall = 0u; s_bin = 0u; s_need_in = 0u; s_members = 0u; }
#pragma unroll
  for (int u = 0; u < EPT; ++u)
    cand[u] = (uint32_t)u * FIN_THREADS + tid < m ? (fine_bin(sc0[u], lo) << TOKEN_BITS) | (uint32_t)ix0[u] : NONE;
  if (ROUNDS == 2) {
    float sc[EPT];
    int32_t ix[EPT];
#pragma unroll
    for (int u = 0; u < EPT; ++u) {
      const uint32_t c = (uint32_t)(EPT + u) * FIN_THREADS + tid;
      sc[u] = c < m ? __ldcg(cs + c) : 0.0f;
      ix[u] = c < m ? __ldcg(ci + c) : 0;
    }
#pragma unroll
    for (int u = 0; u < EPT; ++u)
      cand[EPT + u] = (uint32_t)(EPT + u) * FIN_THREADS + tid < m ? (fine_bin(sc[u], lo) << TOKEN_BITS) | (uint32_t)ix[u] : NONE;
  }
  const uint32_t need0 = min(want, m);
#pragma unroll
  for (int u = 0; u < ROUNDS * EPT; ++u)                      // (s_fine was cleared before the wait)
    if (cand[u] != NONE) atomicAdd(&s_fine[cand[u] >> TOKEN_BITS], 1u);
  __syncthreads();
  uint32_t fh[FPT], local = 0;
#pragma unroll
  for (int x = 0; x < FPT; ++x) {                             // descending: the block prefix is a suffix count
    fh[x] = s_fine[FINE_BINS - 1 - (FPT * tid + x)];
    local += fh[x];
  }
  uint32_t total;
  const uint32_t above = block_exclusive_scan(local, s_warp, &total);
  if (need0 > 0 && need0 < m && above < need0 && above + local >= need0) {
    uint32_t run = above;
#pragma unroll
    for (int x = 0; x < FPT; ++x) {
      if (run < need0 && run + fh[x] >= need0) {
        s_bin = (uint32_t)(FINE_BINS - 1 - (FPT * tid + x));
        s_need_in = need0 - run;
        s_members = fh[x];
      }
      run += fh[x];
    }
  }
  __syncthreads();
  const uint32_t members = s_members, need_in = s_need_in;
  const bool ranked = need0 > 0 && need0 < m && need_in != members;       // bin b is split: its members are ranked
  if (ranked && members > (uint32_t)SMALL) return false;
  // ---- candidates whose bin reaches take_from are chosen outright; the members of a split bin are listed (their
  //      scores are read again: a few dozen loads per head)
  const uint32_t take_from = need0 == 0 ? (uint32_t)FINE_BINS : (need0 >= m ? 0u : (ranked ? s_bin + 1u : s_bin));
  const uint32_t split_bin = ranked ? s_bin : NONE;
#pragma unroll
  for (int u = 0; u < ROUNDS * EPT; ++u) {
    if (cand[u] != NONE) {
      const uint32_t fb = cand[u] >> TOKEN_BITS, t = cand[u] & ((1u << TOKEN_BITS) - 1u);
      if (fb >= take_from) choose(t);
      else if (fb == split_bin) {
        const uint32_t pos = atomicAdd(&s_nsmall, 1u);
        if (pos < (uint32_t)SMALL) s_small[pos] = (((uint64_t)ordered_key(__ldcg(cs + (uint32_t)u * FIN_THREADS + tid))) << 32) | (uint32_t)~t;
      }
    }
  }
  __syncthreads();
  if (ranked) {                                               // a warp per member, its lanes over the others
    const int lane = tid & 31, warp = tid >> 5;
    for (uint32_t i = warp; i < members; i += FIN_THREADS / 32) {
      const uint64_t mine = s_small[i];
      uint32_t larger = 0;
      for (uint32_t j = lane; j < members; j += 32) larger += s_small[j] > mine;
      larger = __reduce_add_sync(0xffffffffu, larger);
      if (lane == 0 && larger < need_in) choose(~(uint32_t)mine);
    }
  }
  __syncthreads();
  // ---- my part's chosen tokens in ascending order: a thread reads its own U groups; its place is the chosen tokens
  //      before the part (counted by all threads) plus those of the threads before it
  uint32_t own = 0;
#pragma unroll
  for (int j = 0; j < FAST_MAXU; ++j)
    if ((uint32_t)j < U) {
      const uint4 x = s_bits4[group_at(U * tid + j)];
      own += __popc(x.x) + __popc(x.y) + __popc(x.z) + __popc(x.w);
    }
  uint32_t totals;                                            // low half: prefix of own; high half: sum of below (both <= 16384)
  const uint32_t prefix = block_exclusive_scan(own | (below << 16), s_warp, &totals);
  const uint32_t n_sink = (uint32_t)F.sink_end, n_loc = (uint32_t)(n - F.local_begin), cnt = need0;
  uint32_t pos = (totals >> 16) + (prefix & 0xffffu);
#pragma unroll
  for (int j = 0; j < FAST_MAXU; ++j)
    if ((uint32_t)j < U) {
      const uint4 x = s_bits4[group_at(U * tid + j)];
      const uint32_t word[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t w = word[q];
        while (w) {
          const uint32_t b = (uint32_t)__ffs((int)w) - 1u;
          w &= w - 1u;
          if (pos < cnt) out[n_sink + pos] = (int32_t)(first_token + ((U * tid + j) << 7) + (q << 5) + b);
          ++pos;
        }
      }
    }
  if (part != 0) return true;
  for (uint32_t e = tid; e < n_sink; e += FIN_THREADS) out[e] = (int32_t)e;
  for (uint32_t e = tid; e < n_loc; e += FIN_THREADS) out[n_sink + cnt + e] = (int32_t)(F.local_begin + e);
  const uint32_t filled = n_sink + cnt + n_loc;
  if (filled != (uint32_t)k) {                                // short selection (non-finite scores)
    if (tid == 0) atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
    for (uint32_t e = filled + tid; e < (uint32_t)k; e += FIN_THREADS) out[e] = (int32_t)(n - 1);   // pad with the last token
  }
  return true;
}

template <int SMALL>
__device__ __forceinline__ bool select_by_fine_histogram(
    const float* __restrict__ cs, const int32_t* __restrict__ ci, long long capacity, const uint32_t* __restrict__ count_ptr,
    bool must_reach_want, uint32_t want, const uint32_t* __restrict__ lo_ptr, long long n, int k, int part,
    Forced F, unsigned char* s_dyn, uint32_t* s_fine, uint32_t* s_warp, int32_t* __restrict__ out, uint32_t* __restrict__ dev_status) {
  // ---- all loads in flight together (the candidate loads are speculative: the list's length is not known yet)
  const int tid = threadIdx.x;
  const uint32_t listed = __ldcg(count_ptr);
  const float lo = __uint_as_float(__ldcg(lo_ptr));
  float sc[FAST_EPT];
  int32_t ix[FAST_EPT];
#pragma unroll
  for (int u = 0; u < FAST_EPT; ++u) {
    const long long c = (long long)u * FIN_THREADS + tid;
    sc[u] = c < capacity ? __ldcg(cs + c) : 0.0f;
    ix[u] = c < capacity ? __ldcg(ci + c) : 0;
  }
  const uint32_t m = (uint32_t)min((long long)listed, capacity);
  if (must_reach_want && listed < want) return false;          // (all conditions are the same for every thread)
  if (m <= (uint32_t)(FAST_EPT * FIN_THREADS))
    return select_by_fine_histogram_rounds<SMALL, 1>(cs, ci, m, sc, ix, want, lo, n, k, part, F, s_dyn, s_fine, s_warp, out, dev_status);
  if (m <= (uint32_t)(2 * FAST_EPT * FIN_THREADS))
    return select_by_fine_histogram_rounds<SMALL, 2>(cs, ci, m, sc, ix, want, lo, n, k, part, F, s_dyn, s_fine, s_warp, out, dev_status);
  return false;
}

// DIRECT = false: candidates are the tokens of the threshold bin (their 12 leading key bits agree), scores are read
//                  from the dense score rows, the number needed comes from the histogram state; the chosen tokens are
//                  OR-ed into the bitmap the filter started, and topk_emit_kernel writes the indices.
// DIRECT = true : candidates are (score, token) pairs collected above a threshold; `want_direct` of them are needed,
//                  the whole 64-bit composite takes part in the select, and the kernel itself writes the head's k
//                  indices in ascending order: the chosen tokens are gathered in shared memory, distributed over
//                  SORT_BUCKETS equal token ranges (counting sort), and ranked inside their range by comparison.
constexpr int SORT_BUCKETS = 4096;
template <bool DIRECT>
__global__ void __launch_bounds__(FIN_THREADS)
topk_select_kernel(const float* __restrict__ scores, long long n, long long score_stride, Forced F,
                   const uint32_t* __restrict__ state, const int32_t* __restrict__ cand,
                   uint32_t* __restrict__ bitmap, long long bitmap_words, int k, int32_t* __restrict__ idx_out,
                   uint32_t* __restrict__ dev_status, uint32_t* __restrict__ tile_count, int ntiles,
                   const uint32_t* __restrict__ cand_count, long long cand_capacity, uint32_t want_direct, int bucket_shift,
                   Gate gate, const float* __restrict__ collect_scores, long long collect_stride, float* __restrict__ collect_score_out,
                   int32_t* __restrict__ collect_idx_out, int cache_entries, int lo_word, int parts, const uint32_t* __restrict__ cand_count_second) {
  constexpr int DIGIT_BITS = 11, DIGITS = 1 << DIGIT_BITS;    // radix of the candidate select
  constexpr int DPT = DIGITS / FIN_THREADS;                    // digits per thread in the suffix scan
  static_assert(FIN_THREADS == 1024, "one pair of s_diff words per lane; digits and ranges per thread");
  static_assert(DIGITS == FINE_BINS, "the short way counts its fine histogram in s_hist");
  constexpr int SMALL_BUCKET = 256;                           // a chosen bucket this small is finished by ranking its members
  __shared__ __align__(8) uint32_t s_hist[DIGITS];            // (also: the members of a small bucket, as 64-bit composites)
  __shared__ uint32_t s_warp[33];
  __shared__ uint32_t s_diff[2 * (FIN_THREADS / 32)];
  __shared__ uint64_t s_prefix;                               // decided leading bits of the threshold composite
  __shared__ uint32_t s_need, s_bucket, s_ntok, s_nsmall;
  extern __shared__ __align__(16) unsigned char s_dyn[];      // composite cache; DIRECT: + range counters, chosen tokens, tokens by range
  uint64_t* s_comp = reinterpret_cast<uint64_t*>(s_dyn);                        // [cache_entries]
  uint32_t* s_range = reinterpret_cast<uint32_t*>(s_comp + cache_entries);      // [SORT_BUCKETS]
  int32_t* s_tok = reinterpret_cast<int32_t*>(s_range + SORT_BUCKETS);          // [k]
  int32_t* s_sorted = s_tok + k;                                                // [k]
  // `parts` CTAs per head: 1, or FAST_PARTS when the short way (select_by_fine_histogram) may apply
  const int head = blockIdx.x / parts, part = blockIdx.x % parts, tid = threadIdx.x;
  const bool counted = DIRECT && parts == FAST_PARTS;
  if (DIRECT) {                                               // shared memory only: done while the previous kernel still runs
    if (counted) {
      const uint32_t G = (uint32_t)fast_select_groups(n) * FIN_THREADS;
      for (uint32_t w = tid; w < G + (G >> 3); w += FIN_THREADS) reinterpret_cast<uint4*>(s_dyn)[w] = make_uint4(0u, 0u, 0u, 0u);
      for (int d = tid; d < DIGITS; d += FIN_THREADS) s_hist[d] = 0u;
    } else
      for (int d = tid; d < SORT_BUCKETS; d += FIN_THREADS) s_range[d] = 0u;
  }
  FATHOM_PDL_WAIT();                                          // the candidates come from the previous kernel
  FATHOM_PDL_RELEASE();                                       // the attention that follows may become resident now
  // gate mode 3: one launch serves both attempts of the fused path - the first attempt's lists if every head holds what
  // it needs, else the lists the second filtering scan has written over them (counted in cand_count_second; their
  // threshold was a bin, so the general way)
  bool second = false;
  if (gate.mode == 3) {
    bool ok = true;
    for (int h = tid; h < gate.heads; h += FIN_THREADS) ok = ok && (__ldcg(gate.counts + h) >= gate.want);
    second = __syncthreads_and(ok) == 0;
  } else if (!fathom_gate_open(gate)) {
    return;
  }
  if (second) cand_count = cand_count_second;
  if (counted) {
    if (!second &&
        select_by_fine_histogram<SMALL_BUCKET>(scores + (size_t)head * (size_t)cand_capacity, cand + (size_t)head * (size_t)cand_capacity,
                                               cand_capacity, cand_count + head, gate.mode == 5 && collect_scores != nullptr, want_direct,
                                               state + head * 8 + lo_word, n, k, part, F, s_dyn, s_hist, s_warp,
                                               idx_out + (size_t)head * k, dev_status))
      return;
    if (part != 0) return;                                    // the general way is one CTA's work
    __syncthreads();                                          // the general way: its range counters lie where the bitmap was
    for (int d = tid; d < SORT_BUCKETS; d += FIN_THREADS) s_range[d] = 0u;
  }
  // dense: scores row of the head, candidate tokens [n];  direct: candidate scores and tokens [cand_capacity]
  // (when the CTA collects its own candidates they are read back through the pointers they were written through)
  const bool own_list = DIRECT && collect_scores != nullptr &&
                        (gate.mode == 5 && __ldcg(gate.counts + head) < gate.want);   // the same for every thread of the CTA
  const float* row = (own_list ? collect_score_out : scores) + (size_t)head * (size_t)(DIRECT ? cand_capacity : score_stride);
  const int32_t* cand_h = (own_list ? collect_idx_out : cand) + (size_t)head * (size_t)(DIRECT ? cand_capacity : n);
  uint32_t* bm = DIRECT ? nullptr : bitmap + (size_t)head * (size_t)bitmap_words;
  uint32_t* tc = DIRECT ? nullptr : tile_count + (size_t)head * ntiles;
  // Second attempt of the single-pass top-k for this head alone (its estimate was too high): the CTA itself collects
  // the head's tokens above the BOUND bin (state word 3) from the score row, replacing the head's candidate list.
  __shared__ uint32_t s_collected;
  if (own_list) {
    if (tid == 0) s_collected = 0u;
    __syncthreads();
    const float lo = edge_of_bin(state[head * 8 + 3]);
    const float* srow = collect_scores + (size_t)head * (size_t)collect_stride;
    float* cs = collect_score_out + (size_t)head * (size_t)cand_capacity;
    int32_t* ci = collect_idx_out + (size_t)head * (size_t)cand_capacity;
    for (long long base = 0; base < n; base += (long long)FIN_THREADS * 4 * 4) {   // uniform trip count: ballots inside
      float4 x[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const long long i = base + ((long long)u * FIN_THREADS + tid) * 4;
        x[u] = i < n ? __ldg(reinterpret_cast<const float4*>(srow + i)) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const long long i = base + ((long long)u * FIN_THREADS + tid) * 4;
        const float e[4] = {x[u].x, x[u].y, x[u].z, x[u].w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const long long t = i + c;
          const bool take = t < n && t >= F.sink_end && t < F.local_begin && e[c] >= lo;
          const unsigned tm = __ballot_sync(0xffffffffu, take);
          if (tm) {
            uint32_t pos = 0;
            const int leader = __ffs(tm) - 1;
            if ((tid & 31) == leader) pos = atomicAdd(&s_collected, (uint32_t)__popc(tm));
            pos = __shfl_sync(0xffffffffu, pos, leader) + __popc(tm & ((1u << (tid & 31)) - 1u));
            if (take && (long long)pos < cand_capacity) { cs[pos] = e[c]; ci[pos] = (int32_t)t; }
          }
        }
      }
    }
    __threadfence_block();
    __syncthreads();
  }
  const uint32_t m = DIRECT ? (uint32_t)min((long long)(own_list ? s_collected : cand_count[head]), cand_capacity)
                            : state[head * 8 + 4];
  const uint32_t need0 = min(DIRECT ? want_direct : state[head * 8 + 2], m);
  constexpr int TOP = DIRECT ? 64 : 52;                       // undecided bits of the composite
  auto composite = [&](uint32_t c) -> uint64_t {
    if (DIRECT) return (((uint64_t)ordered_key(row[c])) << 32) | (uint32_t)(~(uint32_t)cand_h[c]);
    return composite52(row, cand_h[c]);
  };
  // The working set is either all m candidates in global memory or a subset kept in shared memory: everything when
  // m fits, otherwise the bucket of the first digit once it fits (what ranks above that bucket is taken at once).
  __shared__ uint32_t s_ncache;
  bool cached = m <= (uint32_t)cache_entries;
  uint32_t mc = m;                                            // size of the working set
  // Called by all 32 lanes of a warp together; `take` says whether this lane's composite is chosen.
  auto mark = [&](bool take, uint64_t comp) {                 // the token sits in the low 32 bits of every composite
    const int32_t i = (int32_t)~(uint32_t)comp;
    if (DIRECT) {                                             // warp-aggregated append to the list of chosen tokens
      const unsigned tm = __ballot_sync(0xffffffffu, take);
      if (tm) {
        uint32_t pos = 0;
        const int leader = __ffs(tm) - 1;
        if ((tid & 31) == leader) pos = atomicAdd(&s_ntok, (uint32_t)__popc(tm));
        pos = __shfl_sync(0xffffffffu, pos, leader) + __popc(tm & ((1u << (tid & 31)) - 1u));
        if (take && pos < (uint32_t)k) s_tok[pos] = i;
      }
    } else if (take) {
      atomicOr(&bm[bitmap_word(i)], bitmap_bit(i));
      atomicAdd(&tc[i / FILT_TILE], 1u);
    }
  };
  if (tid == 0) { s_ntok = 0u; s_nsmall = 0u; }
  const bool from_cache = DIRECT && cached;                   // every candidate sits in shared memory from the start
  uint64_t first = 0;                                         // a member of the set, the same for every thread
  if (cached && m > 0) {
    // batches of 8 per thread so that a batch's loads are in flight together; on the way: the bits in which any
    // candidate differs from the first one
    first = composite(0);
    uint64_t diff = 0;
    for (uint32_t c0 = 0; c0 < m; c0 += FIN_THREADS * 8) {
      uint64_t comp[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t c = c0 + u * FIN_THREADS + tid;
        comp[u] = c < m ? composite(c) : first;
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const uint32_t c = c0 + u * FIN_THREADS + tid;
        if (c < m) s_comp[c] = comp[u];
        diff |= comp[u] ^ first;
      }
    }
    const uint32_t dlo = __reduce_or_sync(0xffffffffu, (uint32_t)diff), dhi = __reduce_or_sync(0xffffffffu, (uint32_t)(diff >> 32));
    if ((tid & 31) == 0) { s_diff[2 * (tid >> 5)] = dlo; s_diff[2 * (tid >> 5) + 1] = dhi; }
  }
  __syncthreads();

  // ---- radix select of the need0 largest composites among the m candidates: 11-bit digits from the top
  //      undecided bit downwards (the last digit is shorter) until the chosen bucket is taken whole.
  uint64_t thr = 0;                                           // chosen candidates: composite >= thr
  if (need0 > 0 && need0 < m) {
    int hi = TOP;
    uint64_t common = 0;                                      // leading bits shared by every candidate
    if (cached) {
      // All candidates lie in a narrow band of scores, so their leading bits agree: a digit taken there would put
      // every candidate in one histogram bin (thousands of atomics on one address).  Start below the highest bit in
      // which any two composites differ.
      const uint32_t dlo = __reduce_or_sync(0xffffffffu, s_diff[2 * (tid & 31)]);       // (32 warps: one pair of words per lane)
      const uint32_t dhi = __reduce_or_sync(0xffffffffu, s_diff[2 * (tid & 31) + 1]);
      const uint64_t diff = ((uint64_t)dhi << 32) | dlo;
      hi = 64 - __clzll((long long)diff);                     // diff != 0: composites are distinct and m > 1
      if (hi > TOP) hi = TOP;
      common = hi >= 64 ? 0ull : (first >> hi) << hi;
    }
    if (tid == 0) { s_prefix = common; s_need = need0; s_ncache = 0u; }
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
      if (cached && s_bucket <= (uint32_t)SMALL_BUCKET) {
        // a handful of candidates share the chosen digit: list them, rank each against the others, and the one of rank
        // s_need is the threshold itself (composites are distinct)
        uint64_t* s_small = reinterpret_cast<uint64_t*>(s_hist);
        const uint64_t pfx = s_prefix;
        const uint32_t needed = s_need, members = s_bucket;
        for (uint32_t c = tid; c < mc; c += FIN_THREADS) {
          const uint64_t comp = s_comp[c];
          if ((comp >> hi) == (pfx >> hi)) s_small[atomicAdd(&s_nsmall, 1u)] = comp;    // hi < 64 here: a digit has been taken
        }
        __syncthreads();
        if ((uint32_t)tid < members) {
          const uint64_t mine = s_small[tid];
          uint32_t larger = 0;
          for (uint32_t j = 0; j < members; ++j) larger += s_small[j] > mine;
          if (larger + 1u == needed) s_prefix = mine;
        }
        __syncthreads();
        break;
      }
      if (!cached && s_bucket <= (uint32_t)cache_entries) {
        // the undecided bucket fits in shared memory: pull it in, take what ranks above it, go on from there
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
            mark(c < mc && top > ptop, comp[u]);
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
  if (need0 > 0 && !from_cache) {                             // (from the cache the chosen go straight to the counting sort)
    if (DIRECT && cached) {
      // chosen tokens -> list: the warp counts its chosen candidates over all its rounds first and reserves their
      // places with ONE atomic (an atomic per round would serialise the rounds on its return value)
      constexpr int ROUNDS = FIN_CACHE_MAX / FIN_THREADS;      // 16: a cached working set has at most that many rounds
      uint32_t before = 0, mine = 0;                          // chosen by lower lanes / by this lane, over the rounds
      unsigned takes = 0;
#pragma unroll
      for (int r = 0; r < ROUNDS; ++r) {
        if ((uint32_t)(r * FIN_THREADS) >= mc) break;         // (uniform)
        const uint32_t c = r * FIN_THREADS + tid;
        const bool take = c < mc && (need0 >= m || s_comp[c] >= thr);
        const unsigned tm = __ballot_sync(0xffffffffu, take);
        before += __popc(tm & ((1u << (tid & 31)) - 1u));
        mine += take;
        takes |= (unsigned)take << r;
      }
      // lane's first place = warp base + (chosen by lower lanes in all rounds) + ... : order inside the warp's slice is
      // lane-major, any order will do (the list is sorted afterwards)
      uint32_t warp_total = before + mine;                    // at lane 31: the warp's total
      warp_total = __shfl_sync(0xffffffffu, warp_total, 31);
      uint32_t base = 0;
      if ((tid & 31) == 0 && warp_total) base = atomicAdd(&s_ntok, warp_total);
      base = __shfl_sync(0xffffffffu, base, 0) + before;
#pragma unroll
      for (int r = 0; r < ROUNDS; ++r) {
        if ((takes >> r) & 1u) {
          if (base < (uint32_t)k) s_tok[base] = (int32_t)~(uint32_t)s_comp[r * FIN_THREADS + tid];
          ++base;
        }
      }
    } else {
      for (uint32_t c0 = 0; c0 < mc; c0 += FIN_THREADS) {     // uniform trip count: mark is a warp-wide call
        const uint32_t c = c0 + tid;
        const uint64_t comp = c < mc ? (cached ? s_comp[c] : composite(c)) : 0ull;
        mark(c < mc && (need0 >= m || comp >= thr), comp);
      }
    }
  }

  if (DIRECT) {
    // ---- ascending output: sink tokens, the chosen tokens in token order, local tokens
    // (the range counters were cleared at the start; chosen: the need0 largest composites = those that reach thr)
    const bool chosen_all = need0 >= m;
    if (!from_cache) __syncthreads();                         // the list of chosen tokens and its length are complete
    const uint32_t listed = from_cache ? 0u : min(s_ntok, (uint32_t)k);
    if (from_cache) {
      if (need0 > 0)
        for (uint32_t c = tid; c < m; c += FIN_THREADS) {
          const uint64_t comp = s_comp[c];
          if (chosen_all || comp >= thr) atomicAdd(&s_range[(~(uint32_t)comp) >> bucket_shift], 1u);
        }
    } else {
      for (uint32_t e = tid; e < listed; e += FIN_THREADS) atomicAdd(&s_range[(uint32_t)s_tok[e] >> bucket_shift], 1u);
    }
    __syncthreads();
    uint32_t cnt;                                             // chosen tokens = need0
    {                                                         // exclusive prefix over the ranges, in place
      constexpr int RPT = SORT_BUCKETS / FIN_THREADS;
      uint32_t c[RPT], local = 0;
#pragma unroll
      for (int x = 0; x < RPT; ++x) { c[x] = s_range[RPT * tid + x]; local += c[x]; }
      uint32_t run = block_exclusive_scan(local, s_warp, &cnt);
#pragma unroll
      for (int x = 0; x < RPT; ++x) { s_range[RPT * tid + x] = run; run += c[x]; }
      cnt = min(cnt, (uint32_t)k);
    }
    __syncthreads();
    if (from_cache) {                                         // afterwards s_range[r] is the END of range r
      if (need0 > 0)
        for (uint32_t c = tid; c < m; c += FIN_THREADS) {
          const uint64_t comp = s_comp[c];
          if (chosen_all || comp >= thr) {
            const uint32_t t = ~(uint32_t)comp;
            const uint32_t pos = atomicAdd(&s_range[t >> bucket_shift], 1u);
            if (pos < (uint32_t)k) s_sorted[pos] = (int32_t)t;
          }
        }
    } else {
      for (uint32_t e = tid; e < listed; e += FIN_THREADS) {
        const int32_t t = s_tok[e];
        s_sorted[atomicAdd(&s_range[(uint32_t)t >> bucket_shift], 1u)] = t;
      }
    }
    __syncthreads();
    int32_t* out = idx_out + (size_t)head * k;
    const uint32_t n_sink = (uint32_t)F.sink_end, n_loc = (uint32_t)(n - F.local_begin);
    for (uint32_t e0 = 0; e0 < cnt; e0 += FIN_THREADS * 4) {  // four tokens per thread at a time: their loads overlap
      int32_t t[4];
      uint32_t beg[4], end[4], rank[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t e = e0 + u * FIN_THREADS + tid;
        t[u] = e < cnt ? s_sorted[e] : 0;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t r = (uint32_t)t[u] >> bucket_shift;
        beg[u] = r ? s_range[r - 1] : 0u;
        end[u] = s_range[r];
        rank[u] = 0;
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const uint32_t e = e0 + u * FIN_THREADS + tid;
        if (e < cnt) {
          for (uint32_t j = beg[u]; j < end[u]; ++j) rank[u] += s_sorted[j] < t[u];
          out[n_sink + beg[u] + rank[u]] = t[u];
        }
      }
    }
    for (uint32_t e = tid; e < n_sink; e += FIN_THREADS) out[e] = (int32_t)e;
    for (uint32_t e = tid; e < n_loc; e += FIN_THREADS) out[n_sink + cnt + e] = (int32_t)(F.local_begin + e);
    const uint32_t filled = n_sink + cnt + n_loc;
    if (filled != (uint32_t)k) {                              // short selection (non-finite scores)
      if (tid == 0) atomicOr(dev_status, FATHOM_DEV_TOPK_SHORT);
      for (uint32_t e = filled + tid; e < (uint32_t)k; e += FIN_THREADS) out[e] = (int32_t)(n - 1);   // pad with the last token
    }
    return;
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

// Rank in a sample of n_sample of n tokens whose score is, with a margin of four standard deviations of the
// sampling count, low enough that `want` tokens of the whole sequence reach it.
static uint32_t estimate_rank(uint32_t want, long long n_sample, long long n) {
  const double expect = (double)want * (double)n_sample / (double)n;
  return (uint32_t)(expect + 4.0 * sqrt(expect) + 16.0);
}

static bool force_two_pass() {
  static const bool v = [] { const char* e = getenv("FATHOM_TOPK_PATH"); return e && strcmp(e, "two_pass") == 0; }();
  return v;
}

// Whether a row of n scores is selected in a single pass (and with which estimated sample rank).
static bool single_pass_plan(long long n, int k, uint32_t want, uint32_t* rank_out) {
  const long long chunks = n / 1024, sampled = (chunks + 15) / 16;           // whole chunks; chunks 0, 16, 32, .. are sampled
  const long long n_sample = sampled * 1024;
  const uint32_t rank = estimate_rank(want, n_sample, n) + (uint32_t)(k - want);
  *rank_out = rank;
  return !force_two_pass() && want >= 256 && chunks >= 64 && (long long)rank * 8 <= n_sample && (long long)k * 2 <= n_sample;
}

// log2 of the token range per counting-sort bucket of the direct select: the smallest that maps n tokens to SORT_BUCKETS
static int bucket_shift_for(long long n) {
  int s = 0;
  while (((n - 1) >> s) >= SORT_BUCKETS) ++s;
  return s;
}

static size_t select_cache_smem() { return (size_t)FIN_CACHE * 8; }
// composite cache of the direct select: as many entries as k leaves room for in 216 KB, in steps of 1024, at most 16384
static int direct_cache_entries(int k) {
  long long room = (216LL * 1024 - (long long)SORT_BUCKETS * 4 - 2LL * k * 4) / 8;
  room = room / 1024 * 1024;
  return (int)(room > FIN_CACHE_MAX ? FIN_CACHE_MAX : (room < 1024 ? 1024 : room));
}
static size_t direct_select_smem(int k) { return (size_t)direct_cache_entries(k) * 8 + (size_t)SORT_BUCKETS * 4 + (size_t)2 * k * 4; }

// The two attempts of a sampled path on the candidates collected above the estimated bin (counts in S.cand_count)
// and above the bound bin (S.cand_count2): the first runs if every head collected `want`, the second otherwise.
// gate_mode 3: both attempts of the fused path in one launch (after both filtering scans): the first lists if every head
// collected `want`, else the second.
// gate_mode 0: a single attempt whose threshold is a bound (candidates counted in S.cand_count); 1 / 2: first and second
// attempt of the fused path (all heads together, second list counted in S.cand_count2); 5: the single-pass top-k, head
// by head in one launch - a head that collected too few collects again itself, above the bound bin, from `scores`.
static int launch_direct_select(fathom_ctx* ctx, long long n, int Hq, int k, Forced F, uint32_t want, const fathom_topk_scratch& S,
                                int32_t* idx, int gate_mode, cudaStream_t st, const float* scores = nullptr, long long score_stride = 0) {
  static bool attr_set[64] = {};
  if (ctx->device >= 0 && ctx->device < 64 && !attr_set[ctx->device]) {
    FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(topk_select_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 216 * 1024));
    attr_set[ctx->device] = true;
  }
  Gate g = {S.cand_count, want, Hq, gate_mode};
  const int lo_word = gate_mode == 2 ? -1 : 6;                // state word with the score the candidates had to reach (-1: a bin, no short way)
  const size_t smem = direct_select_smem(k);
  // the short way: a known score threshold, tokens that fit in 21 bits, a part's bitmap within the shared memory
  const bool counted = lo_word >= 0 && n <= FAST_MAX_TOKENS && fast_select_groups(n) <= FAST_MAXU && (size_t)fast_select_bytes(n) <= smem;
  const int parts = counted ? FAST_PARTS : 1;
  FATHOM_CUDA_TRY(ctx, fathom_launch_dependent(
      topk_select_kernel<true>, dim3(Hq * parts), dim3(FIN_THREADS), smem, st, (const float*)S.cand_score, n, 0LL, F,
      (const uint32_t*)S.state, (const int32_t*)S.cand, (uint32_t*)nullptr, 0LL, k, idx, ctx->dev_status, (uint32_t*)nullptr, 0,
      (const uint32_t*)(gate_mode == 2 ? S.cand_count2 : S.cand_count), n, want, bucket_shift_for(n), g,
      (const float*)(gate_mode == 5 ? scores : nullptr), score_stride, S.cand_score, S.cand, direct_cache_entries(k), lo_word, parts, (const uint32_t*)(gate_mode == 3 ? S.cand_count2 : nullptr)));
  return FATHOM_OK;
}

static int run_dense_topk(fathom_ctx* ctx, const float* scores, long long n, long long score_stride, int Hq, int k,
                          Forced F, uint32_t want, const fathom_topk_scratch& S, int32_t* idx, cudaStream_t st) {
  const int ntiles = (int)((n + FILT_TILE - 1) / FILT_TILE);
  dim3 fgrid((unsigned)ntiles, (unsigned)Hq);
  Gate always = {nullptr, 0u, 0, 0};
  // Single pass when the row is long enough to estimate the threshold from every 16th 1024-score chunk.
  const long long chunks = n / 1024, sampled = (chunks + 15) / 16;           // whole chunks; chunks 0, 16, 32, .. are sampled
  uint32_t rank = 0;
  const bool single = single_pass_plan(n, k, want, &rank);
  // histograms, per-head states and candidate counters are contiguous at the start of the arena; the sample
  // kernel keeps its histogram in shared memory
  // (the sample kernel writes every state word that path reads and clears the candidate counter: nothing to clear then)
  if (!(single && sampled <= 256)) FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.bitmap - (char*)S.hist, st));
  if (!single) {
    // two passes: histogram of all scores and threshold bin, filter, select within the bin, ascending emission
    const int htile = hist_tile_for(n, Hq);
    dim3 hgrid((unsigned)((n + htile - 1) / htile), (unsigned)Hq);
    topk_hist_kernel<<<hgrid, HIST_THREADS, 0, st>>>(scores, n, score_stride, F, S.hist, S.state, want, ctx->dev_status, htile,
                                                     (long long)htile, 1, 0u);
    topk_filter_kernel<<<fgrid, FILT_THREADS, 0, st>>>(scores, n, score_stride, F, S.state, S.cand, S.bitmap, S.bitmap_words,
                                                       S.tile_count);
    static bool attr_set[64] = {};
    if (ctx->device >= 0 && ctx->device < 64 && !attr_set[ctx->device]) {
      FATHOM_CUDA_TRY(ctx, cudaFuncSetAttribute(topk_select_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                (int)select_cache_smem()));
      attr_set[ctx->device] = true;
    }
    topk_select_kernel<false><<<Hq, FIN_THREADS, select_cache_smem(), st>>>(scores, n, score_stride, F, S.state, S.cand, S.bitmap,
                                                                            S.bitmap_words, k, idx, ctx->dev_status, S.tile_count,
                                                                            ntiles, nullptr, 0, 0u, 0, always, nullptr, 0, nullptr, nullptr, FIN_CACHE,
                                                                            -1, 1, nullptr);
    topk_emit_kernel<<<fgrid, FILT_TILE / 128, 0, st>>>(S.bitmap, S.bitmap_words, S.tile_count, n, k, idx);
  } else {
    // the sample histogram counts forced tokens too, so both ranks allow for all of them: at least k sampled tokens
    // reach the bound bin, hence at least k - forced = want eligible ones
    if (sampled <= 256) {                                              // up to 4M scores per row: one CTA per head
      FATHOM_CUDA_TRY(ctx, fathom_launch_dependent(topk_sample_kernel, dim3(Hq * SAMPLE_CLUSTER), dim3(SAMPLE_THREADS), 0, st, scores, sampled, 16 * 1024LL, score_stride, S.state, rank, (uint32_t)k,
                                                        S.cand_count, (uint32_t*)nullptr));
    } else {
      const int reps = 8;                                              // sampled chunks per CTA
      dim3 sgrid((unsigned)((sampled + reps - 1) / reps), (unsigned)Hq);
      topk_hist_kernel<<<sgrid, HIST_THREADS, 0, st>>>(scores, n, score_stride, F, S.hist, S.state, rank, nullptr, 1024, 16 * 1024LL,
                                                       reps, (uint32_t)k);
    }
    const unsigned ty = (unsigned)(ntiles < 65535 ? ntiles : 65535);
    const dim3 cgrid((unsigned)Hq, ty, (unsigned)((ntiles + ty - 1) / ty));
    if (sampled <= 256) {
      // programmatic dependent launch: the collection's CTAs become resident and load their scores while the 32 CTAs of
      // the sample kernel work; they wait for its completion (griddepcontrol.wait) before they read the threshold
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = cgrid;
      cfg.blockDim = dim3(FILT_THREADS);
      cfg.dynamicSmemBytes = 0;
      cfg.stream = st;
      cudaLaunchAttribute attr[1];
      attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      attr[0].val.programmaticStreamSerializationAllowed = 1;
      cfg.attrs = attr;
      cfg.numAttrs = 1;
      FATHOM_CUDA_TRY(ctx, cudaLaunchKernelEx(&cfg, topk_collect_kernel, scores, n, score_stride, F, (const uint32_t*)S.state,
                                              S.cand_score, S.cand, S.cand_count, ntiles));
    } else {
      topk_collect_kernel<<<cgrid, FILT_THREADS, 0, st>>>(scores, n, score_stride, F, S.state, S.cand_score, S.cand, S.cand_count, ntiles);
    }
    // one launch serves both outcomes: a head whose estimate was low enough selects among its collected candidates; a
    // head that fell short collects above the bound bin itself (one CTA streaming its row) and selects among those
    int rc = launch_direct_select(ctx, n, Hq, k, F, want, S, idx, 5, st, scores, score_stride);
    if (rc != FATHOM_OK) return rc;
  }
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

extern "C" int fathom_topk_passes(const fathom_layout* L, int k, int n_sink, int n_local) {
  if (fathom_check_layout(L) != FATHOM_OK || k < 1 || k > L->n || n_sink < 0 || n_local < 0) return FATHOM_ERR_INVALID_ARG;
  const long long n = L->n;
  const long long sink_end = n_sink < n ? n_sink : n;
  const long long local_begin = (n - n_local > sink_end) ? (n - n_local) : sink_end;
  const long long n_forced = sink_end + (n - local_begin);
  if (n_forced > k) return FATHOM_ERR_INVALID_ARG;
  uint32_t rank;
  return single_pass_plan(n, k, (uint32_t)(k - n_forced), &rank) ? 1 : 2;
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

  // ---- thresholds from a histogram of the sample.  Bound: the bin in which the sample's k-th largest score lies; at
  //      least k tokens of the sample, hence at least k - n_forced eligible tokens of the sequence, reach its lower
  //      edge, so no winner can lie below it.  Estimate: the bin of the rank that `want` tokens of the whole sequence
  //      are expected to reach (plus four standard deviations); far fewer candidates, but no guarantee.
  const long long sampled = (ntiles_scan + step - 1) / step;
  const long long last_start = (sampled - 1) * step * tile;
  const long long n_sample = (sampled - 1) * tile + ((n - last_start) < tile ? (n - last_start) : tile);
  const bool one_cta_sample = n_sample % 1024 == 0 && n_sample / 1024 <= 256;   // whole chunks, up to 4M tokens
  if (!one_cta_sample) FATHOM_CUDA_TRY(ctx, cudaMemsetAsync(S.hist, 0, (char*)S.bitmap - (char*)S.hist, st));
  Forced none;
  none.sink_end = 0;
  none.local_begin = n_sample;
  const uint32_t rank = estimate_rank(want, n_sample, n) + (uint32_t)n_forced;
  const bool two_attempts = !force_two_pass() && want >= 256 && (long long)rank * 2 <= k;
  if (one_cta_sample) {                                       // one CTA per head, histogram in shared memory only
    FATHOM_CUDA_TRY(ctx, fathom_launch_dependent(topk_sample_kernel, dim3(Hq * SAMPLE_CLUSTER), dim3(SAMPLE_THREADS), 0, st, (const float*)S.sample,
                                                 n_sample / 1024, 1024LL, S.sample_stride, S.state, two_attempts ? rank : (uint32_t)k,
                                                 two_attempts ? (uint32_t)k : 0u, S.cand_count, S.cand_count2));
  } else {
    const int htile = hist_tile_for(n_sample, Hq);
    dim3 hgrid((unsigned)((n_sample + htile - 1) / htile), (unsigned)Hq);
    topk_hist_kernel<<<hgrid, HIST_THREADS, 0, st>>>(S.sample, n_sample, S.sample_stride, none, S.hist, S.state,
                                                     two_attempts ? rank : (uint32_t)k, two_attempts ? nullptr : ctx->dev_status,
                                                     htile, (long long)htile, 1, two_attempts ? (uint32_t)k : 0u);
  }
  // ---- full scan that keeps only the tokens reaching their head's threshold, then the exact selection among them
  fathom_scan_fuse fz = {};
  fz.tile_step = 1;
  fz.state = S.state + 6;                                     // the (refined) score threshold of the first attempt
  fz.state_is_score = 1;
  fz.sink_end = F.sink_end;
  fz.local_begin = F.local_begin;
  fz.cand_score = S.cand_score;
  fz.cand_idx = S.cand;
  fz.cand_count = S.cand_count;
  fz.capacity = n;
  fz.gate = fathom_gate{nullptr, 0u, 0, 0};
  rc = fathom_launch_scan_filter(L, planes, scales, q, depth, heads_per_plan, fz, st);
  if (rc != FATHOM_OK) return rc;
  if (two_attempts) {                                         // stands by: runs only if some head's estimate was too high
    fz.state = S.state + 3;
    fz.state_is_score = 0;
    fz.cand_count = S.cand_count2;
    fz.gate = fathom_gate{S.cand_count, want, Hq, 2};
    rc = fathom_launch_scan_filter(L, planes, scales, q, depth, heads_per_plan, fz, st);
    if (rc != FATHOM_OK) return rc;
  }
  // one selection serves both outcomes (a kernel in the chain costs 2.5 us even when it has nothing to do)
  rc = launch_direct_select(ctx, n, Hq, k, F, want, S, idx, two_attempts ? 3 : 0, st);
  if (rc != FATHOM_OK) return rc;
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
