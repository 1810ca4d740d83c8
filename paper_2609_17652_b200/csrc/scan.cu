// fathom_scan: variable-depth bit-plane key scan (Sec. 3.2 prefix dequantiser, Sec. 3.3).
//
// A t-plane read of channel j dequantises to  a * sum_{p<t} (2 b_p - 1) 2^-(p+1)  with a = 8 s the
// block range, so a score is a signed sum of per-(block, channel, plane) weights
//     w[beta][j][p][h] = q_hj * a_{beta,j} * 2^-(p+1),      score_i = sum_rows (b_i ? +w : -w).
// One add per (token, row, head) makes the scan arithmetic-bound (Sec. 6 "Arithmetic per byte"), so the
// kernel trades adds for table lookups: the active (channel, plane) rows of a plan are taken four at a
// time, and for every (64-token block, group of four rows) the 16 possible signed sums are tabulated once
// (15 adds per head) and then looked up per token with the token's four plane bits as the index.
//
// A CTA owns one plan (NH query heads that share the planes read) and 16 blocks (1024 tokens).  Up to 48
// rows at a time it stages, with 16-byte loads, the rows' plane words (128 contiguous bytes per row: every
// row is one contiguous run, Sec. 3.5) and fp16 scales (32 bytes per row) in shared memory; all these loads
// are issued before anything waits, which is what a store in pinned host memory needs to run at link rate.
// Then each of the four warps owns four consecutive blocks (256 tokens) and runs on its own (only
// __syncwarp), walking the staged rows in chunks of four groups.  Per chunk a warp builds its
//   tables     lane (group, head pair, block) takes the four staged scales, forms the weights and writes the
//              16-entry table (8 bytes per entry = two heads); tables are 136 bytes apart so that the 32 lanes
//              store to distinct banks;
//   indices    lane (group, block, half) turns four 32-token row words into 32 four-bit indices with a
//              4 x 4 bit-block transpose across the four registers (20 logic operations);
// and then looks up: lane l owns tokens l and l + 32 of a block: one 8-byte load of the packed indices, then per
//              head pair one 8-byte table load (all lanes hit one 128-byte table: conflict-free) and one
//              packed add.
// Only planes p < t_j and the scales of active channels are ever read.
#include "fathom_common.cuh"

namespace {

constexpr int SCAN_WARPS = 4;
constexpr int SCAN_THREADS = SCAN_WARPS * 32;
constexpr int WB = 4;                                        // blocks per warp
constexpr int TILE_BLOCKS = SCAN_WARPS * WB;                 // 1024 tokens per CTA
constexpr int ROWS_PER_GROUP = 4;
constexpr int GC = 4;                                        // groups per chunk
constexpr int CHUNK_ROWS = GC * ROWS_PER_GROUP;              // 16
constexpr int STAGE_ROWS = 3 * CHUNK_ROWS;                   // rows staged per CTA pass (a B = 48 plan in one pass)

template <int NH> struct ScanCfg {
  static constexpr int HP = NH == 1 ? 1 : NH / 2;            // head pairs (tables per block and group)
  static constexpr int EB = NH == 1 ? 4 : 8;                 // bytes per table entry
  static constexpr int TSTRIDE = 16 * EB + EB;               // bytes between tables (padded: 34 or 17 words)
  static constexpr int NTAB = GC * HP * WB;                  // tables per warp and chunk
};

__device__ __forceinline__ void add2(unsigned long long& acc, unsigned long long v) {
  asm("add.f32x2 %0, %0, %1;" : "+l"(acc) : "l"(v));
}

// 4 x 4 bit-block transpose across four words: afterwards nibble k of word w holds, for token 4 k + w,
// the bits of rows a, b, c, d at bit 0, 1, 2, 3.
__device__ __forceinline__ void transpose_rows(uint32_t& a, uint32_t& b, uint32_t& c, uint32_t& d) {
  uint32_t t;
  t = ((a >> 1) ^ b) & 0x55555555u; b ^= t; a ^= t << 1;
  t = ((c >> 1) ^ d) & 0x55555555u; d ^= t; c ^= t << 1;
  t = ((a >> 2) ^ c) & 0x33333333u; c ^= t; a ^= t << 2;
  t = ((b >> 2) ^ d) & 0x33333333u; d ^= t; b ^= t << 2;
}

// fp32 value whose order-preserving integer image (see topk.cu) has `bin` as its 12 leading bits and zeros below:
// the lower edge of that histogram bin
__device__ __forceinline__ float bin_lower_edge(uint32_t bin) {
  if (bin >= FATHOM_TOPK_BINS) return __uint_as_float(0x7fc00000u);   // past the last bin: nothing reaches it (NaN compares false)
  if (bin <= 7u) return -INFINITY;                                    // bins below -inf's hold no finite score: everything reaches them
  const uint32_t key = bin << 20;
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// first fp16 of staged row r in the padded scale array
__device__ __forceinline__ int scale_offset(int r) { return r * TILE_BLOCKS + (r >> 2) * 8; }

template <int NH>
struct alignas(16) WarpSmem {
  using C = ScanCfg<NH>;
  uint32_t idx[GC][WB * 4 * 2 + 2];                          // [group][(block, token mod 4, half)] + 2 pad words: 8 nibbles each;
                                                             // the pad spreads the four groups over different banks
  alignas(8) unsigned char tab[C::NTAB * C::TSTRIDE];
};

// MODE 0: scores of every token are written (fathom_scan).
// MODE 1: only every tile_step-th tile is scanned and its scores are written compactly (tile i of the launch at
//         token positions 1024 i ..) - the sample from which fathom_scan_topk derives a safe threshold.
// MODE 2: every tile is scanned, nothing is written but the tokens whose score reaches the head's threshold:
//         (score, token) pairs appended to the head's candidate list.
// bx: the CTA's tile (of the launch, or of its item in a batched launch); by: its group of NH query heads
template <int NH, int MODE>
__device__ __forceinline__ void
scan_body(const uint64_t* __restrict__ planes, const uint16_t* __restrict__ scales,
          const float* __restrict__ q, const uint8_t* __restrict__ depth, float* __restrict__ scores,
          long long n, long long nb, long long plane_stride, long long scale_stride, long long score_stride,
          int G, int heads_per_plan, const fathom_scan_fuse& fz, const long long bx, const int by) {
  using C = ScanCfg<NH>;
  constexpr int HP = C::HP, EB = C::EB, TSTRIDE = C::TSTRIDE;
  __shared__ uint16_t row_ch[FATHOM_D * FATHOM_NPLANES];      // channel of active row r
  __shared__ uint8_t row_pl[FATHOM_D * FATHOM_NPLANES];       // plane of active row r
  __shared__ int s_nrows;
  __shared__ int warp_tot[4];
  __shared__ float s_q[NH][FATHOM_D];
  __shared__ float s_thr[NH];                                 // MODE 2: score a token must reach, per head
  // Both staged arrays are read by lanes that differ in the group g = (row / 4) mod 4, and rows four apart would fall on
  // the same banks: the plane words of row r sit at block column c ^ 4 g, and the scales of each group of four rows
  // start 16 bytes further on.
  __shared__ alignas(16) uint64_t s_words[STAGE_ROWS][TILE_BLOCKS];   // staged plane words (block columns swizzled)
  __shared__ alignas(16) uint16_t s_scale[STAGE_ROWS * TILE_BLOCKS + (STAGE_ROWS / 4) * 8];   // staged fp16 scales (padded)
  __shared__ float s_qs[STAGE_ROWS][NH];                               // q_hj * 2^(2 - p) per staged row
  __shared__ WarpSmem<NH> s_warp[SCAN_WARPS];

  FATHOM_PDL_WAIT();                                          // depths (and thresholds) come from the previous kernels
  if (MODE == 2 && !fathom_gate_open(fz.gate)) return;         // second attempt of the fused selection: may have nothing to do
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h0 = by * NH;                                      // first of the NH query heads of this CTA
  const int plan = h0 / heads_per_plan;                        // NH divides heads_per_plan: one plan per CTA
  const int kv = h0 / G;

  // ---- active row list of this plan, ordered by channel then plane (thread = channel)
  {
    const int t = depth[(size_t)plan * FATHOM_D + tid];
    int incl = t;                                             // inclusive prefix of depths over channels
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    for (int e = tid; e < NH * FATHOM_D; e += SCAN_THREADS) s_q[e / FATHOM_D][e % FATHOM_D] = q[(size_t)h0 * FATHOM_D + e];
    if (MODE == 2 && tid < NH)                                // fetched now, needed in the epilogue
      s_thr[tid] = fz.state_is_score ? __uint_as_float(fz.state[(h0 + tid) * 8]) : bin_lower_edge(fz.state[(h0 + tid) * 8]);
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    const int start = base + incl - t;
    for (int p = 0; p < t; ++p) { row_ch[start + p] = (uint16_t)tid; row_pl[start + p] = (uint8_t)p; }
    if (tid == FATHOM_D - 1) s_nrows = base + incl;
    __syncthreads();
  }
  const int nrows = s_nrows;

  WarpSmem<NH>& S = s_warp[warp];
  const long long blk0 = bx * (MODE == 1 ? fz.tile_step : 1) * TILE_BLOCKS;  // first block of this CTA
  const int nblk_cta = (int)min((long long)TILE_BLOCKS, nb - blk0);
  const int wb0 = warp * WB;                                   // first block of this warp within the tile
  const int nblk = max(0, min(WB, nblk_cta - wb0));

  // lookup role: lane owns tokens lane (low word half) and lane + 32 (high half) of each of the warp's blocks
  const int my_w = lane & 3;                                  // word of the transposed quadruple that holds my token
  const int rot = (4 * (lane >> 2) - (EB == 8 ? 3 : 2)) & 31; // brings my nibble to the byte-offset position
  constexpr uint32_t OFFMASK = 15u * EB;
  unsigned long long acc2[WB][2][HP];                         // packed head pairs (NH >= 2)
  float acc1[WB][2];                                          // NH == 1
#pragma unroll
  for (int b = 0; b < WB; ++b)
#pragma unroll
    for (int x = 0; x < 2; ++x) {
      acc1[b][x] = 0.0f;
#pragma unroll
      for (int hp = 0; hp < HP; ++hp) acc2[b][x][hp] = 0ull;
    }

  const uint64_t* planes_kv = planes + (size_t)kv * FATHOM_D * FATHOM_NPLANES * (size_t)plane_stride + blk0;
  const uint16_t* scales_kv = scales + (size_t)kv * FATHOM_D * (size_t)scale_stride + blk0;

  for (int s0 = 0; s0 < nrows; s0 += STAGE_ROWS) {
    const int sc = min(STAGE_ROWS, nrows - s0);                // rows staged in this pass
    if (s0 > 0) __syncthreads();                               // every warp is done with the previous pass
    // ---- stage plane words (8 x 16 B per row), scales (2 x 16 B per row) and per-row query factors
    {
      uint4 wv[STAGE_ROWS * 8 / SCAN_THREADS];
#pragma unroll
      for (int k = 0; k < STAGE_ROWS * 8 / SCAN_THREADS; ++k) {
        const int e = tid + k * SCAN_THREADS, r = e >> 3, c = e & 7;
        wv[k] = make_uint4(0u, 0u, 0u, 0u);
        if (r < sc && 2 * c < nblk_cta) {
          const int j = row_ch[s0 + r], p = row_pl[s0 + r];
          wv[k] = __ldg(reinterpret_cast<const uint4*>(planes_kv + ((size_t)j * FATHOM_NPLANES + p) * (size_t)plane_stride + 2 * c));
        }
      }
      uint4 sv = make_uint4(0u, 0u, 0u, 0u);
      if (tid < STAGE_ROWS * 2) {
        const int r = tid >> 1, c = tid & 1;
        if (r < sc && 8 * c < nblk_cta)
          sv = __ldg(reinterpret_cast<const uint4*>(scales_kv + (size_t)row_ch[s0 + r] * (size_t)scale_stride + 8 * c));
      }
      if (tid < STAGE_ROWS) {
        const bool valid = tid < sc;
        const int j = valid ? row_ch[s0 + tid] : 0, p = valid ? row_pl[s0 + tid] : 0;
        const float pw = valid ? __int_as_float((129 - p) << 23) : 0.0f;   // 8 * 2^-(p+1) = 2^(2-p), exact
#pragma unroll
        for (int h = 0; h < NH; ++h) s_qs[tid][h] = s_q[h][j] * pw;
      }
#pragma unroll
      for (int k = 0; k < STAGE_ROWS * 8 / SCAN_THREADS; ++k) {
        const int e = tid + k * SCAN_THREADS;
        const int r = e >> 3;
        *reinterpret_cast<uint4*>(&s_words[r][(2 * (e & 7)) ^ (((r >> 2) & 3) << 2)]) = wv[k];
      }
      if (tid < STAGE_ROWS * 2) *reinterpret_cast<uint4*>(&s_scale[scale_offset(tid >> 1) + 8 * (tid & 1)]) = sv;
    }
    __syncthreads();

    for (int r0 = 0; r0 < sc; r0 += CHUNK_ROWS) {
      const int rc = min(CHUNK_ROWS, sc - r0);                   // rows in this chunk
      const int gc = (rc + ROWS_PER_GROUP - 1) / ROWS_PER_GROUP; // groups in this chunk (the last may be padded)

      // ---- tables: lane = (group, head pair, block)
#pragma unroll
      for (int t0 = 0; t0 < C::NTAB; t0 += 32) {
        const int t = t0 + lane;
        const int beta = t % WB, hp = (t / WB) % HP, g = t / (WB * HP);
        if (t < C::NTAB && g < gc) {
          float wa[ROWS_PER_GROUP], wb[ROWS_PER_GROUP];
#pragma unroll
          for (int x = 0; x < ROWS_PER_GROUP; ++x) {
            const int r = r0 + g * ROWS_PER_GROUP + x;            // staged rows beyond sc carry zero factors
            const float s = __half2float(__ushort_as_half(s_scale[scale_offset(r) + wb0 + beta]));
            if (NH == 1) {
              wa[x] = s_qs[r][0] * s; wb[x] = 0.0f;
            } else {
              const float2 qq = *reinterpret_cast<const float2*>(&s_qs[r][2 * hp]);
              wa[x] = qq.x * s; wb[x] = qq.y * s;
            }
          }
          float ta[16], tb[16];
          ta[0] = -((wa[0] + wa[1]) + (wa[2] + wa[3]));
          tb[0] = -((wb[0] + wb[1]) + (wb[2] + wb[3]));
#pragma unroll
          for (int x = 0; x < ROWS_PER_GROUP; ++x) {
            const float da = 2.0f * wa[x], db = 2.0f * wb[x];
#pragma unroll
            for (int e = 0; e < (1 << x); ++e) { ta[e + (1 << x)] = ta[e] + da; tb[e + (1 << x)] = tb[e] + db; }
          }
          unsigned char* tab = S.tab + t * TSTRIDE;
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            if (NH == 1) reinterpret_cast<float*>(tab)[e] = ta[e];
            else reinterpret_cast<float2*>(tab)[e] = make_float2(ta[e], tb[e]);
          }
        }
      }

      // ---- indices: lane = (group, block, half)
      {
        const int half = lane & 1, beta = (lane >> 1) & 3, g = lane >> 3;
        if (g < gc) {
          const uint32_t* w32 = reinterpret_cast<const uint32_t*>(&s_words[r0 + g * ROWS_PER_GROUP][(wb0 + beta) ^ (g << 2)]) + half;
          uint32_t a = w32[0 * TILE_BLOCKS * 2];
          uint32_t b = w32[1 * TILE_BLOCKS * 2];
          uint32_t c = w32[2 * TILE_BLOCKS * 2];
          uint32_t d = w32[3 * TILE_BLOCKS * 2];
          transpose_rows(a, b, c, d);
          S.idx[g][(beta * 4 + 0) * 2 + half] = a;
          S.idx[g][(beta * 4 + 1) * 2 + half] = b;
          S.idx[g][(beta * 4 + 2) * 2 + half] = c;
          S.idx[g][(beta * 4 + 3) * 2 + half] = d;
        }
      }
      __syncwarp();

      // ---- lookup
#pragma unroll
      for (int b = 0; b < WB; ++b) {
#pragma unroll
        for (int g = 0; g < GC; ++g) {
          if (g < gc) {
            const uint2 nib = *reinterpret_cast<const uint2*>(&S.idx[g][(b * 4 + my_w) * 2]);
            const uint32_t off_lo = __funnelshift_r(nib.x, nib.x, rot) & OFFMASK;
            const uint32_t off_hi = __funnelshift_r(nib.y, nib.y, rot) & OFFMASK;
            const unsigned char* tab = S.tab + ((g * HP) * WB + b) * TSTRIDE;
            if (NH == 1) {
              acc1[b][0] += *reinterpret_cast<const float*>(tab + off_lo);
              acc1[b][1] += *reinterpret_cast<const float*>(tab + off_hi);
            } else {
#pragma unroll
              for (int hp = 0; hp < HP; ++hp) {
                add2(acc2[b][0][hp], *reinterpret_cast<const unsigned long long*>(tab + hp * (WB * TSTRIDE) + off_lo));
                add2(acc2[b][1][hp], *reinterpret_cast<const unsigned long long*>(tab + hp * (WB * TSTRIDE) + off_hi));
              }
            }
          }
        }
      }
      __syncwarp();
    }
  }

  // ---- epilogue
  if (MODE != 2) {
#pragma unroll
    for (int b = 0; b < WB; ++b) {
      if (b < nblk) {
        const long long tok = (blk0 + wb0 + b) * FATHOM_BLOCK + lane;                       // token scanned
        const long long dst = MODE == 1 ? tok - blk0 * FATHOM_BLOCK + bx * (TILE_BLOCKS * FATHOM_BLOCK) : tok;
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          float* row = scores + (size_t)(h0 + h) * (size_t)score_stride;
#pragma unroll
          for (int x = 0; x < 2; ++x) {
            float v;
            if (NH == 1) v = acc1[b][x];
            else v = __uint_as_float((uint32_t)(acc2[b][x][h >> 1] >> ((h & 1) * 32)));
            if (tok + 32 * x < n) row[dst + 32 * x] = v;
          }
        }
      }
    }
  } else {
    // candidates of this warp's 256 tokens, per head, collected in the (now idle) table memory and appended to
    // the head's global list; entry = (score bits, token)
    constexpr int LIST = (int)(sizeof(S.tab) / sizeof(uint2)) / NH;    // entries per head
    uint2* list = reinterpret_cast<uint2*>(S.tab);
    uint32_t* cnt = S.idx[0];                                          // NH counters (index memory is idle too)
    __syncwarp();
    if (lane < NH) cnt[lane] = 0u;
    __syncwarp();
    float thr[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) thr[h] = s_thr[h];
#pragma unroll
    for (int b = 0; b < WB; ++b) {
      if (b < nblk) {
        const long long tok = (blk0 + wb0 + b) * FATHOM_BLOCK + lane;
#pragma unroll
        for (int x = 0; x < 2; ++x) {
          const long long t = tok + 32 * x;
          const bool elig = t < n && t >= fz.sink_end && t < fz.local_begin;
#pragma unroll
          for (int h = 0; h < NH; ++h) {
            float v;
            if (NH == 1) v = acc1[b][x];
            else v = __uint_as_float((uint32_t)(acc2[b][x][h >> 1] >> ((h & 1) * 32)));
            if (elig && v >= thr[h]) {
              const uint32_t p = atomicAdd(&cnt[h], 1u);
              if (p < (uint32_t)LIST) list[h * LIST + p] = make_uint2(__float_as_uint(v), (uint32_t)t);
              else {                                                   // list full: straight to the global list
                const uint32_t gp = atomicAdd(&fz.cand_count[h0 + h], 1u);
                if ((long long)gp < fz.capacity) {
                  fz.cand_score[(size_t)(h0 + h) * fz.capacity + gp] = v;
                  fz.cand_idx[(size_t)(h0 + h) * fz.capacity + gp] = (int32_t)t;
                }
              }
            }
          }
        }
      }
    }
    // one global atomic per (CTA, head): the four warps' counts are summed, the slice is reserved once
    __shared__ uint32_t s_wcnt[SCAN_WARPS][NH], s_cbase[NH];
    __syncwarp();
    if (lane < NH) s_wcnt[warp][lane] = min(cnt[lane], (uint32_t)LIST);
    __syncthreads();
    if (tid < NH) {
      uint32_t tot = 0;
#pragma unroll
      for (int w = 0; w < SCAN_WARPS; ++w) tot += s_wcnt[w][tid];
      s_cbase[tid] = tot ? atomicAdd(&fz.cand_count[h0 + tid], tot) : 0u;
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < NH; ++h) {
      const uint32_t c = s_wcnt[warp][h];
      uint32_t base = s_cbase[h];
      for (int w = 0; w < warp; ++w) base += s_wcnt[w][h];
      for (uint32_t e = lane; e < c; e += 32) {
        const uint2 it = list[h * LIST + e];
        if ((long long)(base + e) < fz.capacity) {
          fz.cand_score[(size_t)(h0 + h) * fz.capacity + base + e] = __uint_as_float(it.x);
          fz.cand_idx[(size_t)(h0 + h) * fz.capacity + base + e] = (int32_t)it.y;
        }
      }
    }
  }
}

template <int NH, int MODE>
__global__ void __launch_bounds__(SCAN_THREADS, 8)              // 64 registers: occupancy matters more than spills here
scan_kernel(const uint64_t* __restrict__ planes, const uint16_t* __restrict__ scales,
            const float* __restrict__ q, const uint8_t* __restrict__ depth, float* __restrict__ scores,
            long long n, long long nb, long long plane_stride, long long scale_stride, long long score_stride,
            int G, int heads_per_plan, fathom_scan_fuse fz) {
  scan_body<NH, MODE>(planes, scales, q, depth, scores, n, nb, plane_stride, scale_stride, score_stride, G, heads_per_plan, fz,
                      (long long)blockIdx.x, (int)blockIdx.y);
}

// ---- several sessions in one launch (fathom_scan_batch): the items' tiles are laid end to end along grid.x
struct ScanBatch {
  static constexpr int MAX_ITEMS = 32;
  const uint64_t* planes[MAX_ITEMS];
  const uint16_t* scales[MAX_ITEMS];
  const float* q[MAX_ITEMS];
  const uint8_t* depth[MAX_ITEMS];
  float* scores[MAX_ITEMS];
  long long n[MAX_ITEMS], plane_stride[MAX_ITEMS], scale_stride[MAX_ITEMS], score_stride[MAX_ITEMS];
  long long tile_end[MAX_ITEMS];                              // tiles of items 0 .. i, inclusive prefix
  int items;
};

template <int NH>
__global__ void __launch_bounds__(SCAN_THREADS, 8)
scan_batch_kernel(const __grid_constant__ ScanBatch B, int G, int heads_per_plan) {
  int it = 0;
  while (it + 1 < B.items && (long long)blockIdx.x >= B.tile_end[it]) ++it;      // uniform over the CTA, at most 31 steps
  const long long bx = (long long)blockIdx.x - (it ? B.tile_end[it - 1] : 0);
  fathom_scan_fuse fz = {};
  fz.tile_step = 1;
  scan_body<NH, 0>(B.planes[it], B.scales[it], B.q[it], B.depth[it], B.scores[it], B.n[it], (B.n[it] + FATHOM_BLOCK - 1) / FATHOM_BLOCK, B.plane_stride[it],
                   B.scale_stride[it], B.score_stride[it], G, heads_per_plan, fz, bx, (int)blockIdx.y);
}

template <int NH, int MODE>
int launch_scan(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                const uint8_t* depth, int heads_per_plan, float* scores, long long score_stride,
                const fathom_scan_fuse& fz, cudaStream_t st) {
  const long long nb = fathom_nblocks(L->n);
  const long long ntiles = (nb + TILE_BLOCKS - 1) / TILE_BLOCKS;
  const long long gx = MODE == 1 ? (ntiles + fz.tile_step - 1) / fz.tile_step : ntiles;
  dim3 grid((unsigned)gx, (unsigned)(L->n_q_heads / NH));
  if (MODE == 0) {                                            // may become resident while fathom_alloc_depth's kernel runs
    if (fathom_launch_dependent(scan_kernel<NH, MODE>, grid, dim3(SCAN_THREADS), 0, st, planes, scales, q, depth, scores, (long long)L->n,
                                (long long)nb, (long long)L->plane_stride_words, (long long)L->scale_stride, score_stride,
                                L->n_q_heads / L->n_kv_heads, heads_per_plan, fz) != cudaSuccess)
      return FATHOM_ERR_CUDA;
    return 0;
  }
  scan_kernel<NH, MODE><<<grid, SCAN_THREADS, 0, st>>>(planes, scales, q, depth, scores, L->n, nb, L->plane_stride_words,
                                                       L->scale_stride, score_stride, L->n_q_heads / L->n_kv_heads,
                                                       heads_per_plan, fz);
  return 0;
}

template <int MODE>
int dispatch_scan(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                  const uint8_t* depth, int heads_per_plan, float* scores, long long score_stride,
                  const fathom_scan_fuse& fz, cudaStream_t st) {
  switch (heads_per_plan) {
    case 1: return launch_scan<1, MODE>(L, planes, scales, q, depth, 1, scores, score_stride, fz, st);
    case 2: return launch_scan<2, MODE>(L, planes, scales, q, depth, 2, scores, score_stride, fz, st);
    case 4: return launch_scan<4, MODE>(L, planes, scales, q, depth, 4, scores, score_stride, fz, st);
    case 8: return launch_scan<4, MODE>(L, planes, scales, q, depth, 8, scores, score_stride, fz, st);   // two CTAs of four heads share a plan
    default: return FATHOM_ERR_UNSUPPORTED;
  }
}

}  // namespace

int fathom_scan_tile_tokens() { return TILE_BLOCKS * FATHOM_BLOCK; }

int fathom_launch_scan_sample(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, float* sample, long long sample_stride,
                              int tile_step, cudaStream_t st) {
  fathom_scan_fuse fz = {};
  fz.tile_step = tile_step;
  return dispatch_scan<1>(L, planes, scales, q, depth, heads_per_plan, sample, sample_stride, fz, st);
}

int fathom_launch_scan_filter(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, const fathom_scan_fuse& fz, cudaStream_t st) {
  return dispatch_scan<2>(L, planes, scales, q, depth, heads_per_plan, nullptr, 0, fz, st);
}

extern "C" int fathom_scan(fathom_ctx* ctx, const fathom_layout* L, const uint64_t* planes, const uint16_t* scales,
                           const float* q, const uint8_t* depth, int heads_per_plan, float* scores, void* stream) {
  if (!ctx || !planes || !scales || !q || !depth || !scores) return FATHOM_ERR_INVALID_ARG;
  int rc = fathom_check_layout(L);
  if (rc != FATHOM_OK) return rc;
  const int G = L->n_q_heads / L->n_kv_heads;
  if (heads_per_plan < 1 || G % heads_per_plan != 0) return FATHOM_ERR_INVALID_ARG;
  if (!fathom_aligned16(planes) || !fathom_aligned16(scales) || !fathom_aligned16(scores)) return FATHOM_ERR_ALIGNMENT;
  fathom_scan_fuse fz = {};
  fz.tile_step = 1;
  rc = dispatch_scan<0>(L, planes, scales, q, depth, heads_per_plan, scores, L->score_stride, fz, static_cast<cudaStream_t>(stream));
  if (rc != FATHOM_OK) return rc;
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}

extern "C" int fathom_scan_batch(fathom_ctx* ctx, const fathom_scan_item* items, int n_items, int heads_per_plan, void* stream) {
  if (!ctx || !items || n_items < 1) return FATHOM_ERR_INVALID_ARG;
  const int Hkv = items[0].layout.n_kv_heads, Hq = items[0].layout.n_q_heads;
  for (int i = 0; i < n_items; ++i) {
    const fathom_scan_item& it = items[i];
    int rc = fathom_check_layout(&it.layout);
    if (rc != FATHOM_OK) return rc;
    if (it.layout.n_kv_heads != Hkv || it.layout.n_q_heads != Hq) return FATHOM_ERR_INVALID_ARG;   // one model, many sessions
    if (!it.planes || !it.scales || !it.q || !it.depth || !it.scores) return FATHOM_ERR_INVALID_ARG;
    if (!fathom_aligned16(it.planes) || !fathom_aligned16(it.scales) || !fathom_aligned16(it.scores)) return FATHOM_ERR_ALIGNMENT;
  }
  const int G = Hq / Hkv;
  if (heads_per_plan < 1 || G % heads_per_plan != 0) return FATHOM_ERR_INVALID_ARG;
  if (heads_per_plan != 1 && heads_per_plan != 2 && heads_per_plan != 4 && heads_per_plan != 8) return FATHOM_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int first = 0; first < n_items; first += ScanBatch::MAX_ITEMS) {       // at most 32 sessions per launch
    ScanBatch B = {};
    B.items = n_items - first < ScanBatch::MAX_ITEMS ? n_items - first : ScanBatch::MAX_ITEMS;
    long long tiles = 0;
    for (int i = 0; i < B.items; ++i) {
      const fathom_scan_item& it = items[first + i];
      B.planes[i] = it.planes; B.scales[i] = it.scales; B.q[i] = it.q; B.depth[i] = it.depth; B.scores[i] = it.scores;
      B.n[i] = it.layout.n; B.plane_stride[i] = it.layout.plane_stride_words; B.scale_stride[i] = it.layout.scale_stride;
      B.score_stride[i] = it.layout.score_stride;
      tiles += (fathom_nblocks(it.layout.n) + TILE_BLOCKS - 1) / TILE_BLOCKS;
      B.tile_end[i] = tiles;
    }
    const int nh = heads_per_plan == 8 ? 4 : heads_per_plan;  // plans of eight heads are served by two CTAs of four
    dim3 grid((unsigned)tiles, (unsigned)(Hq / nh));
    switch (nh) {
      case 1: scan_batch_kernel<1><<<grid, SCAN_THREADS, 0, st>>>(B, G, heads_per_plan); break;
      case 2: scan_batch_kernel<2><<<grid, SCAN_THREADS, 0, st>>>(B, G, heads_per_plan); break;
      default: scan_batch_kernel<4><<<grid, SCAN_THREADS, 0, st>>>(B, G, heads_per_plan); break;
    }
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
