// fathom_scan: variable-depth bit-plane key scan (Sec. 3.2 prefix dequantiser, Sec. 3.3).
//
// A t-plane read of channel j dequantises to  a * sum_{p<t} (2 b_p - 1) 2^-(p+1)  with a = 8 s the
// block range, so a score is a signed sum of per-(block, channel, plane) weights
//     w[beta][j][p][h] = q_hj * a_{beta,j} * 2^-(p+1),      score_i = sum_rows (b_i ? +w : -w)
//                                                                   = -sum_rows w + sum_{rows with b_i = 1} 2 w.
// The first term is a constant of the (block, head); every active (channel, plane) row then costs one predicated
// add per (token, head).  One add per (token, row, head) is what bounds the scan (Sec. 6 "Arithmetic per byte"): at
// 48 rows and 32 heads the plane bytes would take 9 us of HBM time and the adds take 43 us of the fp32 pipe, so the
// kernel is built around instruction issue, not bandwidth.
//
// A tile is 16 blocks (1024 tokens) of one plan (NH query heads that share the planes read).  With the planes in device
// memory the CTAs are persistent: gridDim.x CTAs per plan walk the tiles round-robin, build the plan's list of active rows
// once, and fetch the next tile's plane words and scales with asynchronous copies (cp.async, 16 bytes each: a row's 16
// words are one contiguous 128-byte run, Sec. 3.5) into the second half of a double buffer while they scan the current
// one; that pays at small budgets (40 against 48 us at B = 4) and is neutral at B = 48, where the adds dominate.  With the
// planes in pinned host memory the grid is one CTA per tile, which keeps the requests on the host link sequential.
// Per tile and pass of up to 48 rows:
//   weights    thread (block, rows r = k mod 8) multiplies the staged fp16 scale with the row's query factors
//              q_hj 2^(3-p) and keeps 2 w of (row, block) for the NH heads; the negated half sums give the bases;
//   adds       lane (block of the warp, octet of its tokens) reads ONE byte of the row's plane word - its eight
//              tokens - and the NH weights, and adds them to the accumulators of the tokens whose bit is set
//              (and + setp + NH predicated adds per token).
// Only planes p < t_j and the scales of active channels are ever read.
#include "fathom_common.cuh"

#include <cstdlib>
#include <cstring>

namespace {

constexpr int SCAN_WARPS = 4;
constexpr int SCAN_THREADS = SCAN_WARPS * 32;
constexpr int WB = 4;                                        // blocks per warp
constexpr int TILE_BLOCKS = SCAN_WARPS * WB;                 // 1024 tokens per tile
constexpr int STAGE_ROWS = 48;                               // rows staged per pass (a B = 48 plan in one pass)
constexpr int TOK = 8;                                       // tokens per lane
constexpr int CTAS_PER_SM = 7;

// fp32 value whose order-preserving integer image (see topk.cu) has `bin` as its 12 leading bits and zeros below:
// the lower edge of that histogram bin
__device__ __forceinline__ float bin_lower_edge(uint32_t bin) {
  if (bin >= FATHOM_TOPK_BINS) return __uint_as_float(0x7fc00000u);   // past the last bin: nothing reaches it (NaN compares false)
  if (bin <= 7u) return -INFINITY;                                    // bins below -inf's hold no finite score: everything reaches them
  const uint32_t key = bin << 20;
  return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
}

// a[h] += w[h] for the NH heads if bit MASK of `bits` is set.  (A predicated add.f32x2 is not issued as one
// instruction, so the adds are scalar.)
template <int MASK>
__device__ __forceinline__ void add_if(float (&a)[4], uint32_t bits, const float (&w)[4]) {
  asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %4, %5;\n\tsetp.ne.u32 p, t, 0;\n\t@p add.f32 %0, %0, %6;\n\t@p add.f32 %1, %1, %7;\n\t"
      "@p add.f32 %2, %2, %8;\n\t@p add.f32 %3, %3, %9;\n\t}"
      : "+f"(a[0]), "+f"(a[1]), "+f"(a[2]), "+f"(a[3]) : "r"(bits), "n"(MASK), "f"(w[0]), "f"(w[1]), "f"(w[2]), "f"(w[3]));
}
template <int MASK>
__device__ __forceinline__ void add_if(float (&a)[2], uint32_t bits, const float (&w)[2]) {
  asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %2, %3;\n\tsetp.ne.u32 p, t, 0;\n\t@p add.f32 %0, %0, %4;\n\t@p add.f32 %1, %1, %5;\n\t}"
      : "+f"(a[0]), "+f"(a[1]) : "r"(bits), "n"(MASK), "f"(w[0]), "f"(w[1]));
}
template <int MASK>
__device__ __forceinline__ void add_if(float (&a)[1], uint32_t bits, const float (&w)[1]) {
  asm("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\tand.b32 t, %1, %2;\n\tsetp.ne.u32 p, t, 0;\n\t@p add.f32 %0, %0, %3;\n\t}"
      : "+f"(a[0]) : "r"(bits), "n"(MASK), "f"(w[0]));
}

// NH consecutive floats as one shared-memory access
__device__ __forceinline__ void load_heads(const float* p, float (&v)[4]) {
  const float4 x = *reinterpret_cast<const float4*>(p); v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
}
__device__ __forceinline__ void load_heads(const float* p, float (&v)[2]) {
  const float2 x = *reinterpret_cast<const float2*>(p); v[0] = x.x; v[1] = x.y;
}
__device__ __forceinline__ void load_heads(const float* p, float (&v)[1]) { v[0] = *p; }
__device__ __forceinline__ void store_heads(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
__device__ __forceinline__ void store_heads(float* p, const float (&v)[2]) { *reinterpret_cast<float2*>(p) = make_float2(v[0], v[1]); }
__device__ __forceinline__ void store_heads(float* p, const float (&v)[1]) { *p = v[0]; }

// 16-byte asynchronous copy global -> shared; `valid` false writes zeros and reads nothing
__device__ __forceinline__ void copy16_async(void* dst, const void* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int bytes = valid ? 16 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void copies_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int PENDING>
__device__ __forceinline__ void copies_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(PENDING) : "memory"); }

// ---- the sessions of one launch: their tiles are laid end to end (fathom_scan has one item)
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
struct alignas(16) ScanSmem {
  uint16_t row_ch[FATHOM_D * FATHOM_NPLANES];                 // channel of active row r
  uint8_t row_pl[FATHOM_D * FATHOM_NPLANES];                  // plane of active row r
  int nrows;
  int warp_tot[4];
  float thr[NH];                                              // MODE 2: score a token must reach, per head
  alignas(16) uint64_t words[2][STAGE_ROWS][TILE_BLOCKS];     // staged plane words, double buffered
  alignas(16) uint16_t scale[2][STAGE_ROWS][TILE_BLOCKS];     // staged fp16 scales, double buffered
  alignas(16) float qs[2 * STAGE_ROWS][NH];                   // q_hj * 2^(3 - p) of every row (plans of up to 96 rows) or of a pass
  alignas(16) float w2[STAGE_ROWS][TILE_BLOCKS][NH];          // 2 w of (row, block, head)
  alignas(16) float pb[SCAN_WARPS][TILE_BLOCKS][NH];          // -sum of w over the rows a warp weighted, per block
  uint32_t cnt[SCAN_WARPS][NH], wcnt[SCAN_WARPS][NH], cbase[NH];   // MODE 2: candidate counters
};

// MODE 0: scores of every token are written (fathom_scan, fathom_scan_batch).
// MODE 1: only every tile_step-th tile is scanned and its scores are written compactly (tile i of the launch at
//         token positions 1024 i ..) - the sample from which fathom_scan_topk derives a safe threshold.
// MODE 2: every tile is scanned, nothing is written but the tokens whose score reaches the head's threshold:
//         (score, token) pairs appended to the head's candidate list.
// grid = (CTAs per plan, groups of NH query heads); MODE 1 and 2 are launched with one item.
template <int NH, int MODE>
__global__ void __launch_bounds__(SCAN_THREADS, CTAS_PER_SM)
scan_kernel(const __grid_constant__ ScanBatch B, int G, int heads_per_plan, fathom_scan_fuse fz) {
  __shared__ ScanSmem<NH> M;
  constexpr int QS_ROWS = (int)(sizeof(M.qs) / sizeof(M.qs[0]));

  FATHOM_PDL_WAIT();                                          // depths (and thresholds) come from the previous kernels
  if (MODE == 2 && !fathom_gate_open(fz.gate)) return;         // second attempt of the fused selection: may have nothing to do
  const int total = (int)B.tile_end[B.items - 1];              // tiles of this launch (tile and block indices fit 32 bits)
  int g = blockIdx.x;                                          // my current tile of the launch
  if (g >= total) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int h0 = blockIdx.y * NH;                              // first of the NH query heads of this CTA
  const int plan = h0 / heads_per_plan;                        // NH divides heads_per_plan: one plan per CTA
  const int kv = h0 / G;
  const int beta = lane >> 3, oct = lane & 7;                  // lane = (block of the warp, octet of its tokens)
  const int myb = warp * WB + beta;                            // my block within the tile
  if (MODE == 2 && tid < NH)                                   // read after the barriers of the first item's row list
    M.thr[tid] = fz.state_is_score ? __uint_as_float(fz.state[(h0 + tid) * 8]) : bin_lower_edge(fz.state[(h0 + tid) * 8]);

  int item = -1, nrows = 0, npass = 1;

  // ---- a new session: the active row list of this plan, ordered by channel then plane (thread = channel), and
  //      the rows' query factors if they all fit
  auto enter_item = [&](int tile) {
    int it = item < 0 ? 0 : item;
    while (tile >= B.tile_end[it]) ++it;                       // uniform over the CTA; items only move forward
    if (it == item) return;
    item = it;
    const int t = B.depth[it][(size_t)plan * FATHOM_D + tid];
    int incl = t;                                              // inclusive prefix of depths over channels
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
    }
    if (lane == 31) M.warp_tot[warp] = incl;
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += M.warp_tot[w];
    const int start = before + incl - t;
    for (int p = 0; p < t; ++p) { M.row_ch[start + p] = (uint16_t)tid; M.row_pl[start + p] = (uint8_t)p; }
    if (tid == FATHOM_D - 1) M.nrows = before + incl;
    __syncthreads();
    nrows = M.nrows;
    npass = nrows > 0 ? (nrows + STAGE_ROWS - 1) / STAGE_ROWS : 1;
    if (nrows <= QS_ROWS && tid < nrows) {                     // made visible by the barrier that precedes the first weights
      const int j = M.row_ch[tid], p = M.row_pl[tid];
      const float pw = __int_as_float((130 - p) << 23);        // 2 * 8 * 2^-(p+1) = 2^(3-p), exact
#pragma unroll
      for (int h = 0; h < NH; ++h) M.qs[tid][h] = __ldg(B.q[it] + (size_t)(h0 + h) * FATHOM_D + j) * pw;
    }
  };

  // first block of launch tile `tile` within its session
  auto first_block = [&](int tile) -> int {
    const int tl = tile - (item ? (int)B.tile_end[item - 1] : 0);
    return tl * (MODE == 1 ? fz.tile_step : 1) * TILE_BLOCKS;
  };

  // ---- asynchronous copies of the plane words (8 x 16 B per row) and scales (2 x 16 B per row) of one pass of a tile
  auto prefetch = [&](int tile, int pass, int buf) {
    const int blk0 = first_block(tile);
    const int nb = (int)((B.n[item] + FATHOM_BLOCK - 1) / FATHOM_BLOCK);
    const int nblk_cta = min(TILE_BLOCKS, nb - blk0);
    const int s0 = pass * STAGE_ROWS, sc = min(STAGE_ROWS, nrows - s0);
    // (strides are below 2^32 elements: one 32 x 32 -> 64-bit multiply per address)
    const uint32_t plane_stride = (uint32_t)B.plane_stride[item], scale_stride = (uint32_t)B.scale_stride[item];
    const uint64_t* planes_kv = B.planes[item] + (uint64_t)(kv * FATHOM_D * FATHOM_NPLANES) * plane_stride + blk0;
    const uint16_t* scales_kv = B.scales[item] + (uint64_t)(kv * FATHOM_D) * scale_stride + blk0;
#pragma unroll
    for (int k = 0; k < STAGE_ROWS * 8 / SCAN_THREADS; ++k) {
      const int e = tid + k * SCAN_THREADS, r = e >> 3, c = e & 7;
      if (r < sc) {
        const uint32_t row = (uint32_t)M.row_ch[s0 + r] * FATHOM_NPLANES + M.row_pl[s0 + r];
        const bool valid = 2 * c < nblk_cta;
        copy16_async(&M.words[buf][r][2 * c], valid ? (const void*)(planes_kv + (uint64_t)row * plane_stride + 2 * c) : (const void*)B.planes[item],
                     valid);
      }
    }
    if (tid < STAGE_ROWS * 2) {
      const int r = tid >> 1, c = tid & 1;
      if (r < sc) {
        const bool valid = 8 * c < nblk_cta;
        copy16_async(&M.scale[buf][r][8 * c],
                     valid ? (const void*)(scales_kv + (uint64_t)M.row_ch[s0 + r] * scale_stride + 8 * c) : (const void*)B.scales[item], valid);
      }
    }
    copies_commit();
  };

  enter_item(g);
  int pass = 0, buf = 0;
  prefetch(g, 0, 0);
  float acc[TOK][NH], base[NH];

  while (true) {
    // ---- the stage after this one: the next pass of the tile, or the first pass of my next tile
    int g_next = g;
    int pass_next = pass + 1;
    if (pass_next == npass) { g_next = g + gridDim.x; pass_next = 0; }
    const bool more = g_next < total;
    const bool same_item = more && g_next < B.tile_end[item];
    if (same_item) {
      prefetch(g_next, pass_next, buf ^ 1);                    // lands while this stage is scanned
      copies_wait<1>();
    } else {
      copies_wait<0>();
    }
    __syncthreads();                                           // this stage's words and scales are in place

    const int s0 = pass * STAGE_ROWS, sc = min(STAGE_ROWS, nrows - s0);
    const int q0 = nrows <= QS_ROWS ? s0 : 0;                  // where this pass's query factors start in M.qs
    if (nrows > QS_ROWS) {                                     // too many rows to keep all factors: those of this pass
      if (tid < sc) {
        const int j = M.row_ch[s0 + tid], p = M.row_pl[s0 + tid];
        const float pw = __int_as_float((130 - p) << 23);
#pragma unroll
        for (int h = 0; h < NH; ++h) M.qs[tid][h] = __ldg(B.q[item] + (size_t)(h0 + h) * FATHOM_D + j) * pw;
      }
      __syncthreads();
    }

    // ---- doubled weights of every (row, block) and the blocks' bases: thread = (block, rows r = k mod 8)
    {
      const int b = tid & 15, k = tid >> 4;
      float pb[NH];
#pragma unroll
      for (int h = 0; h < NH; ++h) pb[h] = 0.0f;
      for (int r = k; r < sc; r += SCAN_THREADS / 16) {
        const float s = __half2float(__ushort_as_half(M.scale[buf][r][b]));
        float w2[NH];
        load_heads(&M.qs[q0 + r][0], w2);
#pragma unroll
        for (int h = 0; h < NH; ++h) { w2[h] *= s; pb[h] += w2[h]; }
        store_heads(&M.w2[r][b][0], w2);
      }
#pragma unroll
      for (int h = 0; h < NH; ++h) pb[h] = -0.5f * (pb[h] + __shfl_xor_sync(0xffffffffu, pb[h], 16));
      if (lane < 16) store_heads(&M.pb[warp][b][0], pb);
    }
    __syncthreads();

    if (pass == 0) {
#pragma unroll
      for (int h = 0; h < NH; ++h) {
        base[h] = 0.0f;
#pragma unroll
        for (int t = 0; t < TOK; ++t) acc[t][h] = 0.0f;
      }
    }
#pragma unroll
    for (int w = 0; w < SCAN_WARPS; ++w) {
      float pb[NH];
      load_heads(&M.pb[w][myb][0], pb);
#pragma unroll
      for (int h = 0; h < NH; ++h) base[h] += pb[h];
    }

    // ---- one predicated add per (token, row, head)
    {
      const unsigned char* my_bytes = reinterpret_cast<const unsigned char*>(&M.words[buf][0][myb]) + oct;
      const float* my_w = &M.w2[0][myb][0];
#pragma unroll 4
      for (int r = 0; r < sc; ++r) {
        const uint32_t bits = my_bytes[r * (TILE_BLOCKS * 8)];
        float w[NH];
        load_heads(my_w + r * (TILE_BLOCKS * NH), w);
        add_if<1>(acc[0], bits, w);
        add_if<2>(acc[1], bits, w);
        add_if<4>(acc[2], bits, w);
        add_if<8>(acc[3], bits, w);
        add_if<16>(acc[4], bits, w);
        add_if<32>(acc[5], bits, w);
        add_if<64>(acc[6], bits, w);
        add_if<128>(acc[7], bits, w);
      }
    }

    if (pass == npass - 1) {
      // ---- scores of my eight tokens: base + what the set bits added
      float v[NH][TOK];
#pragma unroll
      for (int t = 0; t < TOK; ++t)
#pragma unroll
        for (int h = 0; h < NH; ++h) v[h][t] = acc[t][h] + base[h];
      const uint32_t n = (uint32_t)B.n[item];                  // n < 2^31
      const int blk0 = first_block(g);
      const bool have_block = blk0 + myb < (n + FATHOM_BLOCK - 1) / FATHOM_BLOCK;
      const uint32_t tok = (uint32_t)(blk0 + myb) * FATHOM_BLOCK + oct * TOK;                // my first token

      if (MODE != 2) {
        if (have_block) {
          const uint32_t dst = MODE == 1 ? (uint32_t)g * (TILE_BLOCKS * FATHOM_BLOCK) + myb * FATHOM_BLOCK + oct * TOK : tok;
#pragma unroll
          for (int h = 0; h < NH; ++h) {
            float* row = B.scores[item] + (size_t)(h0 + h) * (size_t)B.score_stride[item] + dst;
            if (tok + TOK <= n) {
              *reinterpret_cast<float4*>(row) = make_float4(v[h][0], v[h][1], v[h][2], v[h][3]);
              *reinterpret_cast<float4*>(row + 4) = make_float4(v[h][4], v[h][5], v[h][6], v[h][7]);
            } else {
#pragma unroll
              for (int t = 0; t < TOK; ++t)
                if (tok + t < n) row[t] = v[h][t];
            }
          }
        }
      } else {
        // candidates of this warp's 256 tokens, per head, collected in the (now idle) weight memory and appended to
        // the head's global list; entry = (score bits, token)
        constexpr int LIST = (int)(sizeof(M.w2) / sizeof(uint2)) / SCAN_WARPS / NH;    // entries per warp and head
        __syncthreads();                                                   // every warp is done with the weights
        uint2* list = reinterpret_cast<uint2*>(&M.w2[0][0][0]) + warp * (LIST * NH);
        uint32_t* cnt = M.cnt[warp];
        if (lane < NH) cnt[lane] = 0u;
        __syncwarp();
        if (have_block) {
#pragma unroll
          for (int t = 0; t < TOK; ++t) {
            const long long ti = (long long)tok + t;
            const bool elig = ti < n && ti >= fz.sink_end && ti < fz.local_begin;
#pragma unroll
            for (int h = 0; h < NH; ++h) {
              if (elig && v[h][t] >= M.thr[h]) {
                const uint32_t p = atomicAdd(&cnt[h], 1u);
                if (p < (uint32_t)LIST) list[h * LIST + p] = make_uint2(__float_as_uint(v[h][t]), (uint32_t)ti);
                else {                                                   // list full: straight to the global list
                  const uint32_t gp = atomicAdd(&fz.cand_count[h0 + h], 1u);
                  if ((long long)gp < fz.capacity) {
                    fz.cand_score[(size_t)(h0 + h) * fz.capacity + gp] = v[h][t];
                    fz.cand_idx[(size_t)(h0 + h) * fz.capacity + gp] = (int32_t)ti;
                  }
                }
              }
            }
          }
        }
        // one global atomic per (tile, head): the four warps' counts are summed, the slice is reserved once
        __syncwarp();
        if (lane < NH) M.wcnt[warp][lane] = min(cnt[lane], (uint32_t)LIST);
        __syncthreads();
        if (tid < NH) {
          uint32_t tot = 0;
#pragma unroll
          for (int w = 0; w < SCAN_WARPS; ++w) tot += M.wcnt[w][tid];
          M.cbase[tid] = tot ? atomicAdd(&fz.cand_count[h0 + tid], tot) : 0u;
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < NH; ++h) {
          const uint32_t c = M.wcnt[warp][h];
          uint32_t at = M.cbase[h];
          for (int w = 0; w < warp; ++w) at += M.wcnt[w][h];
          for (uint32_t e = lane; e < c; e += 32) {
            const uint2 it = list[h * LIST + e];
            if ((long long)(at + e) < fz.capacity) {
              fz.cand_score[(size_t)(h0 + h) * fz.capacity + at + e] = __uint_as_float(it.x);
              fz.cand_idx[(size_t)(h0 + h) * fz.capacity + at + e] = (int32_t)it.y;
            }
          }
        }
      }
    }

    if (!more) break;
    __syncthreads();                                           // every warp is done with this stage's buffers
    g = g_next;
    pass = pass_next;
    buf ^= 1;
    if (!same_item) {                                          // first tile of another session: nothing was fetched ahead
      enter_item(g);
      prefetch(g, 0, buf);
    }
  }
}

// Whether the planes are read over the host link (pinned host memory mapped into the device's address space)
static bool planes_in_host_memory(const void* planes) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, planes) != cudaSuccess) { cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost;
}

// CTAs per plan.  Planes in HBM: as many as are resident at once (and no more than there are tiles), each walking
// several tiles.  Planes read over the host link: one CTA per tile, so that CTAs become resident in block order - all
// tiles of one plan before the next plan's - and the link sees a few long sequential streams (48 rows of one KV head)
// instead of eight times as many short ones; the link, not instruction issue, bounds that scan.
static int scan_ctas_per_plan(long long tiles, int plans, bool host_planes) {
  if (const char* e = getenv("FATHOM_SCAN_CTAS_PER_PLAN")) {   // tests and tuning: a fixed number (read at every call)
    const long long v = atoll(e);
    if (v >= 1) return (int)(v < tiles ? v : tiles);
  }
  if (host_planes) return (int)tiles;
  static int sms[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  if (!sms[dev]) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    sms[dev] = v;
  }
  long long x = (long long)sms[dev] * CTAS_PER_SM / plans;
  if (x < 1) x = 1;
  return (int)(x < tiles ? x : tiles);
}

template <int NH, int MODE>
int launch_scan(const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz, bool dependent,
                cudaStream_t st) {
  const long long tiles = B.tile_end[B.items - 1];
  if (tiles <= 0) return FATHOM_OK;
  const int plans = Hq / NH;
  dim3 grid((unsigned)scan_ctas_per_plan(tiles, plans, planes_in_host_memory(B.planes[0])), (unsigned)plans);
  if (dependent) {                                            // may become resident while the previous kernel of the stream runs
    if (fathom_launch_dependent(scan_kernel<NH, MODE>, grid, dim3(SCAN_THREADS), 0, st, B, Hq / Hkv, heads_per_plan, fz) != cudaSuccess)
      return FATHOM_ERR_CUDA;
    return FATHOM_OK;
  }
  scan_kernel<NH, MODE><<<grid, SCAN_THREADS, 0, st>>>(B, Hq / Hkv, heads_per_plan, fz);
  return FATHOM_OK;
}

template <int MODE>
int dispatch_scan(const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz, bool dependent,
                  cudaStream_t st) {
  switch (heads_per_plan) {
    case 1: return launch_scan<1, MODE>(B, Hkv, Hq, 1, fz, dependent, st);
    case 2: return launch_scan<2, MODE>(B, Hkv, Hq, 2, fz, dependent, st);
    case 4: return launch_scan<4, MODE>(B, Hkv, Hq, 4, fz, dependent, st);
    case 8: return launch_scan<4, MODE>(B, Hkv, Hq, 8, fz, dependent, st);   // two CTAs of four heads share a plan
    default: return FATHOM_ERR_UNSUPPORTED;
  }
}

// one session as a batch of one; `tile_step` > 1 lists only the sampled tiles
ScanBatch single_item(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q, const uint8_t* depth,
                      float* scores, long long score_stride, int tile_step) {
  ScanBatch B = {};
  B.items = 1;
  B.planes[0] = planes; B.scales[0] = scales; B.q[0] = q; B.depth[0] = depth; B.scores[0] = scores;
  B.n[0] = L->n; B.plane_stride[0] = L->plane_stride_words; B.scale_stride[0] = L->scale_stride; B.score_stride[0] = score_stride;
  const long long tiles = (fathom_nblocks(L->n) + TILE_BLOCKS - 1) / TILE_BLOCKS;
  B.tile_end[0] = (tiles + tile_step - 1) / tile_step;
  return B;
}

}  // namespace

int fathom_scan_tile_tokens() { return TILE_BLOCKS * FATHOM_BLOCK; }

int fathom_launch_scan_sample(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, float* sample, long long sample_stride,
                              int tile_step, cudaStream_t st) {
  fathom_scan_fuse fz = {};
  fz.tile_step = tile_step;
  return dispatch_scan<1>(single_item(L, planes, scales, q, depth, sample, sample_stride, tile_step), L->n_kv_heads, L->n_q_heads,
                          heads_per_plan, fz, false, st);
}

int fathom_launch_scan_filter(const fathom_layout* L, const uint64_t* planes, const uint16_t* scales, const float* q,
                              const uint8_t* depth, int heads_per_plan, const fathom_scan_fuse& fz, cudaStream_t st) {
  return dispatch_scan<2>(single_item(L, planes, scales, q, depth, nullptr, 0, 1), L->n_kv_heads, L->n_q_heads, heads_per_plan, fz,
                          false, st);
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
  rc = dispatch_scan<0>(single_item(L, planes, scales, q, depth, scores, L->score_stride, 1), L->n_kv_heads, L->n_q_heads, heads_per_plan,
                        fz, true, static_cast<cudaStream_t>(stream));
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
  fathom_scan_fuse fz = {};
  fz.tile_step = 1;
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
    const int rc = dispatch_scan<0>(B, Hkv, Hq, heads_per_plan, fz, false, st);
    if (rc != FATHOM_OK) return rc;
  }
  FATHOM_CUDA_TRY(ctx, cudaGetLastError());
  return FATHOM_OK;
}
