// The scan with one predicated fp32 add per (token, plane bit, head) on the CUDA cores: the first formulation of
// fathom_scan, kept selectable (FATHOM_SCAN_PATH=simt, read once) as a cross-check of the tensor-core kernel in scan.cu.
//
// A t-plane read of channel j dequantises to  a * sum_{p<t} (2 b_p - 1) 2^-(p+1)  with a = 8 s the
// block range (Sec. 3.2), so a score is a signed sum of per-(block, channel, plane) weights
//     w[beta][j][p][h] = q_hj * a_{beta,j} * 2^-(p+1),      score_i = -sum_rows w + sum_{rows with b_i = 1} 2 w.
// The first term is a constant of the (block, head); every active (channel, plane) row then costs one predicated
// add per (token, head) (Sec. 7 "Arithmetic per byte"): 1.6 G adds at n = 1M, B = 48 occupy the fp32 pipes for 43 us,
// which is why this kernel stops at a third of the HBM peak.
//
// A tile is 16 blocks (1024 tokens) of one plan (NH query heads that share the planes read).  With the planes in device
// memory the CTAs are persistent: gridDim.x CTAs per plan walk the tiles round-robin, build the plan's list of active rows
// once, and fetch the next tile's plane words and scales with asynchronous copies (cp.async, 16 bytes each: a row's 16
// words are one contiguous 128-byte run, Sec. 3.6) into the second half of a double buffer while they scan the current
// one.  With the planes in pinned host memory the grid is one CTA per tile, which keeps the requests on the host link sequential.
// Per tile and pass of up to 48 rows:
//   weights    thread (block, rows r = k mod 8) multiplies the staged fp16 scale with the row's query factors
//              q_hj 2^(3-p) and keeps 2 w of (row, block) for the NH heads; the negated half sums give the bases;
//   adds       lane (block of the warp, octet of its tokens) reads ONE byte of the row's plane word - its eight
//              tokens - and the NH weights, and adds them to the accumulators of the tokens whose bit is set
//              (and + setp + NH predicated adds per token).
// Only planes p < t_j and the scales of active channels are ever read.
#include "scan_shared.cuh"

namespace {

constexpr int SCAN_WARPS = 4;
constexpr int SCAN_THREADS = SCAN_WARPS * 32;
constexpr int WB = 4;                                        // blocks per warp
constexpr int TILE_BLOCKS = FATHOM_SCAN_TILE_BLOCKS;          // 1024 tokens per tile = SCAN_WARPS * WB blocks
constexpr int STAGE_ROWS = 48;                               // rows staged per pass (a B = 48 plan in one pass)
constexpr int TOK = 8;                                       // tokens per lane
constexpr int CTAS_PER_SM = 7;

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
scan_simt_kernel(const __grid_constant__ ScanBatch B, int G, int heads_per_plan, fathom_scan_fuse fz) {
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
    M.thr[tid] = fz.state_is_score ? __uint_as_float(fz.state[(h0 + tid) * 8]) : fathom_bin_lower_edge(fz.state[(h0 + tid) * 8]);

  int item = -1, nrows = 0, npass = 1;

  // ---- a new session: the active row list of this plan, ordered by channel then plane (thread = channel), and
  //      the rows' query factors if they all fit
  auto enter_item = [&](int tile) {
    int it = item < 0 ? 0 : item;
    while (tile >= B.tile_end[it]) ++it;                       // uniform over the CTA; items only move forward
    if (it == item) return;
    item = it;
    const int t = min((int)B.depth[it][(size_t)plan * FATHOM_D + tid], FATHOM_NPLANES);   // a depth above 4 (an unwritten buffer) must not index past the row list
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
        fathom_copy_async<16>(&M.words[buf][r][2 * c], valid ? (const void*)(planes_kv + (uint64_t)row * plane_stride + 2 * c) : (const void*)B.planes[item],
                     valid);
      }
    }
    if (tid < STAGE_ROWS * 2) {
      const int r = tid >> 1, c = tid & 1;
      if (r < sc) {
        const bool valid = 8 * c < nblk_cta;
        fathom_copy_async<16>(&M.scale[buf][r][8 * c],
                     valid ? (const void*)(scales_kv + (uint64_t)M.row_ch[s0 + r] * scale_stride + 8 * c) : (const void*)B.scales[item], valid);
      }
    }
    fathom_copies_commit();
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
      fathom_copies_wait<1>();
    } else {
      fathom_copies_wait<0>();
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

template <int NH, int MODE>
int launch_scan(const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz, bool dependent,
                cudaStream_t st) {
  const long long tiles = B.tile_end[B.items - 1];
  if (tiles <= 0) return FATHOM_OK;
  const int plans = Hq / NH;
  dim3 grid((unsigned)fathom_scan_grid_ctas(tiles, plans, fathom_planes_in_host_memory(B.planes[0]), CTAS_PER_SM), (unsigned)plans);
  if (dependent) {                                            // may become resident while the previous kernel of the stream runs
    if (fathom_launch_dependent(scan_simt_kernel<NH, MODE>, grid, dim3(SCAN_THREADS), 0, st, B, Hq / Hkv, heads_per_plan, fz) != cudaSuccess)
      return FATHOM_ERR_CUDA;
    return FATHOM_OK;
  }
  scan_simt_kernel<NH, MODE><<<grid, SCAN_THREADS, 0, st>>>(B, Hq / Hkv, heads_per_plan, fz);
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

}  // namespace

int fathom_scan_simt_dispatch(int mode, const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz,
                              bool dependent, cudaStream_t st) {
  switch (mode) {
    case 0: return dispatch_scan<0>(B, Hkv, Hq, heads_per_plan, fz, dependent, st);
    case 1: return dispatch_scan<1>(B, Hkv, Hq, heads_per_plan, fz, dependent, st);
    case 2: return dispatch_scan<2>(B, Hkv, Hq, heads_per_plan, fz, dependent, st);
    default: return FATHOM_ERR_INVALID_ARG;
  }
}
