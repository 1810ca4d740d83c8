// fathom_scan: variable-depth bit-plane key scan (Sec. 3.2 prefix dequantiser, Sec. 3.3), accumulate on the tensor cores.
//
// A t-plane read of channel j dequantises to  a * sum_{p<t} (2 b_p - 1) 2^-(p+1)  with a = 8 s the block range, so with
// the active (channel, plane) pairs of a plan as "rows" r = (j, p) a score is
//     score[i][h] = sum_r  sigma[i][r] * s[beta(i)][j(r)]  *  q_h,j(r) 2^(2 - p(r)),        sigma = +1 if the bit is set, else -1:
// a [tokens x rows] . [rows x heads] product whose left operand is the stored fp16 scale with the plane bit as its sign
// - exact in fp16 - and whose right operand depends on neither token nor block.  One add per (token, row, head) on the
// CUDA cores is what bounds the scan (Sec. 7 "Arithmetic per byte": 1.6 G adds at n = 1M, B = 48, 43 us of fp32 pipe
// against 9 us of HBM time for the planes); here the adds go to the tensor cores and the CUDA cores only expand the
// plane bits into the left operand, two integer instructions per pair of elements:
//   * left operand (registers): a lane holds, for 8 consecutive tokens of a block (one byte of each plane word) and 4 of
//     every 16 rows, the half2 (s_r, s_r') of a row pair; the element of token i is that pair with the sign bits flipped
//     where the tokens' bits are clear:  pair ^ (~(bytes << shift_i) & 0x80008000);
//   * right operand: q_hj 2^(2-p) / E_h (E_h a power of two near max_j |q_hj|) split into an fp16 head and an fp16 tail
//     scaled by 2^11 (together 22 significant bits + rounding = the precision of an fp32 weight), columns
//     (head, part) = 4 x 2 = the 8 columns of mma.sync.m16n8k16; built once per session and plan in shared memory;
//   * fp16 x fp16 products are exact in the fp32 accumulators; score = E_h (acc_head + 2^-11 acc_tail).  The order of
//     the accumulation is fixed by the row list alone, so scores do not depend on the launch geometry.
// The tcgen05 path was not taken for this contraction: its left operand must sit in shared or tensor memory, i.e. every
// expanded element would be written and read once more (2 bytes per (token, row) against 1/8 byte of plane bits), and
// the expansion, not the multiply-add, is what costs here (12 mma per 64 tokens x 48 rows against ~100 integer ops).
//
// A tile is 16 blocks (1024 tokens) of one plan (NH query heads that share the planes read).  With the planes in device
// memory the CTAs are persistent: gridDim.x CTAs per plan walk the tiles round-robin, build the plan's row list and right
// operand once, and fetch the next stage's plane words and scales with asynchronous copies (cp.async; a row's words are
// one contiguous run, Sec. 3.6) into the other half of a double buffer.  A stage is a sub-tile of TB blocks and up to
// ROWS rows: plans of up to 48 rows take whole tiles (TB = 16: 128-byte runs, a warp owns 4 blocks), up to 96 rows half
// tiles (TB = 8), deeper plans quarter tiles (TB = 4, a warp owns one block and carries its accumulators over passes of
// 160 rows), so that the staging buffers do not grow with the budget.  With the planes in pinned host memory the grid is
// one CTA per tile, which keeps the requests on the host link sequential.
// Only planes p < t_j and the scales of active channels are ever read.
#include "scan_shared.cuh"

#include <cstdlib>
#include <cstring>
#include <type_traits>

namespace {

constexpr int THREADS = 128, WARPS = 4;
constexpr int TILE_BLOCKS = FATHOM_SCAN_TILE_BLOCKS;
constexpr int MAX_ROWS = FATHOM_D * FATHOM_NPLANES;          // 512 (channel, plane) pairs
constexpr int STAGE_KSTEPS = 10;                             // 16 rows per mma; a stage holds at most 160 rows
constexpr int WORD_STAGE_BYTES = 7680;                       // staged plane words of one stage (padded rows)
constexpr int SCALE_STAGE_BYTES = 4608;                      // staged fp16 scales of one stage (padded rows)
#ifndef FATHOM_SCAN_CTAS_PER_SM
#define FATHOM_SCAN_CTAS_PER_SM 4                               // 16 warps per SM with ~115 registers each beat 24 warps with 80
#endif
constexpr int CTAS_PER_SM = FATHOM_SCAN_CTAS_PER_SM;

// Stage geometry for sub-tiles of TB blocks.  The row pitches are padded so that the four lanes of a quad, which read
// rows two apart, hit different banks (plane bytes: pitch / 4 = 4 mod 32 for TB = 16, ...).
template <int TB>
struct Geo {
  static constexpr int ROW_BYTES = 8 * TB + 16;               // pitch of a staged plane-word row
  static constexpr int SCALE_ELEMS = TB == 4 ? 12 : 24;       // pitch of a staged scale row, fp16 elements
  static constexpr int ROWS = TB == 16 ? 48 : TB == 8 ? 96 : 160;   // rows per stage (multiples of 16)
  static_assert(ROWS * ROW_BYTES <= WORD_STAGE_BYTES && ROWS * SCALE_ELEMS * 2 <= SCALE_STAGE_BYTES, "stage buffers too small");
};

// MODE 2.  A lane whose eight scores hold a candidate parks all eight in its warp's ring (three stores, no atomic, no
// loop); when the ring may not take another round of 32, the warp sifts it with all lanes, one parked group per lane,
// into the CTA's four candidate lists (one shared-memory atomic per head); the lists go to the heads' global lists once,
// when the CTA has scanned its last tile (one global atomic per head and CTA).
constexpr int PARK_RING = 64;                                // parked groups per warp
constexpr int CAND_LIST = 256;                               // candidates per head the CTA keeps; beyond that: straight to the global list

template <int MODE>
struct alignas(16) Smem {
  uint16_t row_id[MAX_ROWS];                                  // active row r: channel * 4 + plane
  uint32_t woff[MAX_ROWS];                                    // where its plane words start within the KV head, in 16-byte units
  uint32_t soff[MAX_ROWS];                                    // where its channel's scales start within the KV head, in 16-byte units
  int nrows;
  int warp_tot[WARPS];
  float wmax[WARPS][4];                                       // per warp: max_j |q_hj| of its channels
  float hscale[4], hinv[4];                                   // E_h and 1 / E_h
  float thr[4];                                               // MODE 2: score a token must reach, per head
  uint32_t ccount[4], cbase[4];                               // MODE 2: candidates in the CTA's lists; where they go in the global lists
  uint32_t elig[2];                                           // MODE 2: eligible tokens lo <= t < hi of the session
  alignas(16) float4 park_lo[MODE == 2 ? WARPS * PARK_RING : 1];     // MODE 2: scores 0..3 of a parked group
  alignas(16) float4 park_hi[MODE == 2 ? WARPS * PARK_RING : 1];     //         scores 4..7
  uint32_t park_tok[MODE == 2 ? WARPS * PARK_RING : 1];       //         its first token (30 bits) and the head within the CTA (2 bits)
  uint2 clist[MODE == 2 ? 4 * CAND_LIST : 1];                 // MODE 2: (score bits, token) per head
  alignas(16) uint2 bfr[STAGE_KSTEPS][32];                    // right operand of the rows of a pass: per 16 rows, the two B registers of every lane
  alignas(16) unsigned char words[2][WORD_STAGE_BYTES];       // staged plane words, double buffered
  alignas(16) unsigned char scale[2][SCALE_STAGE_BYTES];      // staged fp16 scales, double buffered
};

// D += A B, A 16 x 16 (row), B 16 x 8 (col), fp16 operands, fp32 accumulators
__device__ __forceinline__ void mma_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// the scale pair with each half's sign flipped where bit (15 - SH) resp. (31 - SH) of `bytes` is clear
template <int SH>
__device__ __forceinline__ uint32_t signed_pair(uint32_t pair, uint32_t bytes) {
  return pair ^ (~(bytes << SH) & 0x80008000u);
}

// eight consecutive scores: one 32-byte store where the address allows it (a whole sector per lane), else two of 16 bytes
__device__ __forceinline__ void store_scores8(float* row, const float (&v)[8]) {
  if ((reinterpret_cast<uintptr_t>(row) & 31u) == 0) {
    asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(row), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]),
                 "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
  } else {
    *reinterpret_cast<float4*>(row) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(row + 4) = make_float4(v[4], v[5], v[6], v[7]);
  }
}

// One block (64 tokens: this lane's eight are byte `wp[0]` of every staged plane word) times the rows of a stage, 16 rows per
// step: the lane's two row pairs of a step are rows 2 t4, 2 t4 + 1 and 2 t4 + 8, 2 t4 + 9 of the sixteen.  NKS > 0: that
// many steps, unrolled (the loads of all steps are in flight at once); NKS = 0: `nks` steps in a loop.
// Slice j of the accumulators: mma row gq = token 8 gq + 2 j, row gq + 8 = token 8 gq + 2 j + 1.
template <int ROW_BYTES, int SCALE_ELEMS, int NKS>
__device__ __forceinline__ void mma_rows(float (&acc)[4][4], const unsigned char* wp, const uint16_t* sp, const uint2* bfr_lane, int nks) {
  auto step = [&](int ks) {
    const uint2 bf = bfr_lane[ks * 32];
    const unsigned char* w = wp + ks * (16 * ROW_BYTES);
    const uint16_t* sc = sp + ks * (16 * SCALE_ELEMS);
    const uint32_t x0 = __byte_perm(w[0], w[ROW_BYTES], 0x5410);
    const uint32_t x1 = __byte_perm(w[8 * ROW_BYTES], w[9 * ROW_BYTES], 0x5410);
    const uint32_t S0 = __byte_perm(sc[0], sc[SCALE_ELEMS], 0x5410);
    const uint32_t S1 = __byte_perm(sc[8 * SCALE_ELEMS], sc[9 * SCALE_ELEMS], 0x5410);
    mma_16816(acc[0], signed_pair<15>(S0, x0), signed_pair<14>(S0, x0), signed_pair<15>(S1, x1), signed_pair<14>(S1, x1), bf.x, bf.y);
    mma_16816(acc[1], signed_pair<13>(S0, x0), signed_pair<12>(S0, x0), signed_pair<13>(S1, x1), signed_pair<12>(S1, x1), bf.x, bf.y);
    mma_16816(acc[2], signed_pair<11>(S0, x0), signed_pair<10>(S0, x0), signed_pair<11>(S1, x1), signed_pair<10>(S1, x1), bf.x, bf.y);
    mma_16816(acc[3], signed_pair<9>(S0, x0), signed_pair<8>(S0, x0), signed_pair<9>(S1, x1), signed_pair<8>(S1, x1), bf.x, bf.y);
  };
  if (NKS > 0) {
#pragma unroll
    for (int ks = 0; ks < NKS; ++ks) step(ks);
  } else {
#pragma unroll 1
    for (int ks = 0; ks < nks; ++ks) step(ks);
  }
}

// MODE 0: scores of every token are written (fathom_scan, fathom_scan_batch).
// MODE 1: only every tile_step-th tile is scanned and its scores are written compactly (tile i of the launch at
//         token positions 1024 i ..) - the sample from which fathom_scan_topk derives a safe threshold.
// MODE 2: every tile is scanned, nothing is written but the tokens whose score reaches the head's threshold:
//         (score, token) pairs appended to the head's candidate list.
// grid = (CTAs per plan, groups of NH query heads); MODE 1 and 2 are launched with one item.
// IN_HBM: every store of the launch lies in device memory (its rows are staged past the L1).
template <int NH, int MODE, bool IN_HBM>
__global__ void __launch_bounds__(THREADS, CTAS_PER_SM)
scan_kernel(const __grid_constant__ ScanBatch B, int G, int heads_per_plan, fathom_scan_fuse fz) {
  extern __shared__ __align__(16) unsigned char scan_smem[];   // sizeof(Smem<MODE>): more than the static limit in MODE 2
  Smem<MODE>& M = *reinterpret_cast<Smem<MODE>*>(scan_smem);

  FATHOM_PDL_WAIT();                                          // depths (and thresholds) come from the previous kernels
  if (MODE == 2 && !fathom_gate_open(fz.gate)) return;         // second attempt of the fused selection: may have nothing to do
  const int total = (int)B.tile_end[B.items - 1];              // tiles of this launch (tile and block indices fit 32 bits)
  int g = blockIdx.x;                                          // my current tile of the launch
  if (g >= total) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr bool in_hbm = IN_HBM;
  const int gq = lane >> 2, t4 = lane & 3;                     // mma fragment coordinates: lane = (row group, column pair)
  const int h0 = blockIdx.y * NH;                              // first of the NH query heads of this CTA
  const int plan = h0 / heads_per_plan;                        // NH divides heads_per_plan: one plan per CTA
  const int kv = h0 / G;
  const int myh = t4 < NH ? t4 : 0;                            // the head whose scores this lane receives (lanes t4 >= NH: none)
  if (MODE == 2 && tid < 4) M.ccount[tid] = 0u;
  if (MODE == 2 && tid == 0) {                                 // (MODE 2 is launched with one session)
    const long long n0 = B.n[0];
    const long long hi = fz.local_begin < n0 ? fz.local_begin : n0, lo = fz.sink_end < hi ? fz.sink_end : hi;
    M.elig[0] = (uint32_t)lo;
    M.elig[1] = (uint32_t)hi;
  }
  if (MODE == 2 && tid < NH)                                   // read after the barriers of the first item's row list
    M.thr[tid] = fz.state_is_score ? __uint_as_float(fz.state[(h0 + tid) * 8]) : fathom_bin_lower_edge(fz.state[(h0 + tid) * 8]);

  int item = -1, nrows = 0, tb = TILE_BLOCKS, rows_stage = Geo<16>::ROWS, npass = 1, nb_item = 0;
  float hs = 1.0f, hs_tail = 0.0f;                             // E of my head and E 2^-11

  // ---- right operand of the rows of pass `pass` (made visible by the barrier that precedes the pass's arithmetic): entry
  //      (kstep, lane, i) holds rows 16 kstep + 2 (lane & 3) + 8 i and the next one of the pass, column lane >> 2 = (head, part)
  auto fill_bfr = [&](int pass) {
    const int s0 = pass * rows_stage, sc = min(rows_stage, nrows - s0);
    const int entries = ((sc + 15) >> 4) * 64;
    for (int e = tid; e < entries; e += THREADS) {
      const int ks = e >> 6, ln = (e >> 1) & 31, i = e & 1;
      const int col = ln >> 2, head = col >> 1, part = col & 1;
      const int r0 = s0 + ks * 16 + 2 * (ln & 3) + 8 * i;
      uint32_t packed = 0u;
      if (head < NH) {
        const float inv = M.hinv[head];
#pragma unroll
        for (int z = 0; z < 2; ++z) {
          const int r = r0 + z;
          float v = 0.0f;
          if (r < nrows) {
            const int id = M.row_id[r];
            v = __ldg(B.q[item] + (size_t)(h0 + head) * FATHOM_D + (id >> 2)) * inv * __int_as_float((129 - (id & 3)) << 23);
          }
          const __half hi = __float2half_rn(v);
          const __half out = part ? __float2half_rn((v - __half2float(hi)) * 2048.0f) : hi;
          packed |= (uint32_t)__half_as_ushort(out) << (16 * z);
        }
      }
      reinterpret_cast<uint32_t*>(&M.bfr[ks][ln])[i] = packed;
    }
  };

  // ---- a new session: the active row list of this plan, ordered by channel then plane (thread = channel), the
  //      heads' power-of-two scales (the right operand of every 16 rows follows once the first stage has been requested)
  auto enter_item = [&](int tile) {
    int it = item < 0 ? 0 : item;
    while (tile >= B.tile_end[it]) ++it;                       // uniform over the CTA; items only move forward
    if (it == item) return;
    item = it;
    nb_item = (int)((B.n[it] + FATHOM_BLOCK - 1) / FATHOM_BLOCK);
    const int t = min((int)B.depth[it][(size_t)plan * FATHOM_D + tid], FATHOM_NPLANES);   // a depth above 4 (an unwritten buffer) must not index past the row list
    int incl = t;                                              // inclusive prefix of depths over channels
    float qa[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) qa[h] = fabsf(__ldg(B.q[it] + (size_t)(h0 + h) * FATHOM_D + tid));
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += y;
#pragma unroll
      for (int h = 0; h < NH; ++h) qa[h] = fmaxf(qa[h], __shfl_xor_sync(0xffffffffu, qa[h], o));
    }
    if (lane == 31) M.warp_tot[warp] = incl;
#pragma unroll
    for (int h = 0; h < NH; ++h)
      if (lane == h) M.wmax[warp][h] = qa[h];
    __syncthreads();
    int before = 0;
    for (int w = 0; w < warp; ++w) before += M.warp_tot[w];
    const int start = before + incl - t;
    const uint32_t half_stride = (uint32_t)(B.plane_stride[it] >> 1), eighth_stride = (uint32_t)(B.scale_stride[it] >> 3);
    for (int p = 0; p < t; ++p) {                              // (511 * half_stride < 2^32: fathom_check_layout)
      M.row_id[start + p] = (uint16_t)(tid * FATHOM_NPLANES + p);
      M.woff[start + p] = (uint32_t)(tid * FATHOM_NPLANES + p) * half_stride;
      M.soff[start + p] = (uint32_t)tid * eighth_stride;
    }
    if (tid == FATHOM_D - 1) M.nrows = before + incl;
    if (tid < NH) {                                            // E = 2^floor(log2 max|q|), kept inside the normal range
      float m = 0.0f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) m = fmaxf(m, M.wmax[w][tid]);
      int eb = (int)(__float_as_uint(m) >> 23);
      eb = eb < 1 ? 1 : (eb > 253 ? 253 : eb);
      M.hscale[tid] = __int_as_float(eb << 23);
      M.hinv[tid] = __int_as_float((254 - eb) << 23);
    }
    __syncthreads();
    nrows = M.nrows;
    if (nrows <= Geo<16>::ROWS) { tb = 16; rows_stage = Geo<16>::ROWS; }
    else if (nrows <= Geo<8>::ROWS) { tb = 8; rows_stage = Geo<8>::ROWS; }
    else { tb = 4; rows_stage = Geo<4>::ROWS; }
    npass = nrows > rows_stage ? (nrows + rows_stage - 1) / rows_stage : 1;
    hs = M.hscale[myh];
    hs_tail = hs * 4.8828125e-4f;                              // 2^-11
  };

  // first block of launch tile `tile` within its session
  auto first_block = [&](int tile) -> int {
    const int tl = tile - (item ? (int)B.tile_end[item - 1] : 0);
    return tl * (MODE == 1 ? fz.tile_step : 1) * TILE_BLOCKS;
  };

  // ---- asynchronous copies of the plane words and scales of one stage: sub-tile u of `tile`, rows of `pass`
  auto prefetch = [&](int tile, int u, int pass, int buf) {
    const int blk0 = first_block(tile) + u * tb;
    const int nblk = min(tb, nb_item - blk0);                  // >= 1: stages past the last block are never entered
    const int s0 = pass * rows_stage, sc = min(rows_stage, nrows - s0);
    // 16-byte units throughout: plane_stride is even, scale_stride a multiple of 8, blk0 a multiple of tb
    const uint4* planes_kv = reinterpret_cast<const uint4*>(B.planes[item]) +
                             (uint64_t)(kv * FATHOM_D * FATHOM_NPLANES) * (uint64_t)(B.plane_stride[item] >> 1) + (blk0 >> 1);
    const unsigned char* scales_kv = reinterpret_cast<const unsigned char*>(B.scales[item]) +
                                     (uint64_t)(kv * FATHOM_D) * (uint64_t)B.scale_stride[item] * 2 + (uint64_t)blk0 * 2;
    const int sh = tb == 16 ? 3 : (tb == 8 ? 2 : 1);           // 16-byte copies per row of plane words: tb / 2
    const int row_bytes = 8 * tb + 16;
    unsigned char* wdst = M.words[buf];
    const int c = tid & ((1 << sh) - 1);                       // my 16-byte column of every row I copy
    const bool valid = 2 * c < nblk;
    for (int r = tid >> sh; r < sc; r += THREADS >> sh)
      fathom_copy_async<16>(wdst + r * row_bytes + c * 16, valid ? planes_kv + M.woff[s0 + r] + c : planes_kv, valid, in_hbm);
    unsigned char* sdst = M.scale[buf];
    if (tb == 16) {
      const int cs = tid & 1;
      const bool vs = 8 * cs < nblk;
      for (int r = tid >> 1; r < sc; r += THREADS >> 1)
        fathom_copy_async<16>(sdst + r * (Geo<16>::SCALE_ELEMS * 2) + cs * 16, vs ? scales_kv + (uint64_t)M.soff[s0 + r] * 16 + cs * 16 : scales_kv, vs,
                              in_hbm);
    } else if (tb == 8) {
      for (int r = tid; r < sc; r += THREADS)
        fathom_copy_async<16>(sdst + r * (Geo<8>::SCALE_ELEMS * 2), scales_kv + (uint64_t)M.soff[s0 + r] * 16, true, in_hbm);
    } else {
      for (int r = tid; r < sc; r += THREADS)
        fathom_copy_async<8>(sdst + r * (Geo<4>::SCALE_ELEMS * 2), scales_kv + (uint64_t)M.soff[s0 + r] * 16, true);
    }
    // rows that pad the last 16: scale 0, so that whatever the stale plane bytes say they contribute +-0
    const int pad = ((sc + 15) & ~15) - sc;
    const int wpr = (tb == 4 ? Geo<4>::SCALE_ELEMS : Geo<16>::SCALE_ELEMS) / 2;   // 32-bit words per scale row
    for (int e = tid; e < pad * wpr; e += THREADS)
      reinterpret_cast<uint32_t*>(sdst)[(sc + e / wpr) * wpr + e % wpr] = 0u;
    fathom_copies_commit();
  };

  float acc[4][4];                                             // [16-token slice of the block][c0..c3]
  uint32_t parked = 0u, stages = 0u;                           // MODE 2: groups in my warp's ring (the same in every lane); stages done

  enter_item(g);
  const float my_thr = MODE == 2 ? M.thr[myh] : 0.0f;
  int u = 0, pass = 0, buf = 0;
  prefetch(g, 0, 0, 0);                                        // the first stage's rows are on their way ...
  fill_bfr(0);                                                 // ... while the right operand is made

  // ---- MODE 2, whole warp: the parked groups, one per lane and round, into the CTA's candidate lists.  A lane marks the
  //      candidates among its group's eight scores (score reaches the head's threshold, token eligible).  Nearly always
  //      there is one: the lanes that have any are ranked per head with a ballot, lanes 0..3 reserve the heads' places
  //      with one shared-memory atomic each, and every such lane writes its first candidate; further candidates of a
  //      group take a place of their own.  All warps of a CTA sift at the same stages (every fourth): a warp that did
  //      it alone would keep the others waiting at the stage barrier.
  auto sift = [&]() {
    if (MODE != 2) return;
    __syncwarp();                                              // the parked groups are visible to the whole warp
    const uint32_t elo = M.elig[0], ehi = M.elig[1];
    auto append = [&](uint32_t h, uint32_t pos, float val, uint32_t token) {
      if (pos < (uint32_t)CAND_LIST) {
        M.clist[h * CAND_LIST + pos] = make_uint2(__float_as_uint(val), token);
      } else {                                                 // list full (only with a threshold far too low): straight to the global list
        const uint32_t at = atomicAdd(&fz.cand_count[h0 + h], 1u);
        if ((long long)at < fz.capacity) {
          fz.cand_score[(size_t)(h0 + h) * fz.capacity + at] = val;
          fz.cand_idx[(size_t)(h0 + h) * fz.capacity + at] = (int32_t)token;
        }
      }
    };
    for (uint32_t e0 = 0; e0 < parked; e0 += 32) {
      const uint32_t e = warp * PARK_RING + e0 + lane;
      const bool mine = e0 + lane < parked;
      const uint32_t tk = mine ? M.park_tok[e] : 0u;
      const uint32_t h = tk >> 30, tok = tk & 0x3fffffffu;
      const float th = M.thr[h];
      uint32_t mask = 0u;
      if (mine) {
        const float4 a = M.park_lo[e], b = M.park_hi[e];
        const float w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
        for (int x = 0; x < 8; ++x) mask |= (w[x] >= th && tok + x - elo < ehi - elo ? 1u : 0u) << x;
      }
      auto score_at = [&](uint32_t x) { return reinterpret_cast<const float*>(x < 4u ? &M.park_lo[e] : &M.park_hi[e])[x & 3u]; };
      uint32_t rank = 0u, tot = 0u, base = 0u;
#pragma unroll
      for (int hh = 0; hh < 4; ++hh) {
        const unsigned with = __ballot_sync(0xffffffffu, mask != 0u && h == (uint32_t)hh);
        if (h == (uint32_t)hh) rank = __popc(with & ((1u << lane) - 1u));
        if (lane == hh) tot = __popc(with);
      }
      if (lane < 4 && tot) base = atomicAdd(&M.ccount[lane], tot);
      base = __shfl_sync(0xffffffffu, base, (int)h);
      if (mask) {
        const uint32_t x = (uint32_t)__ffs((int)mask) - 1u;
        mask &= mask - 1u;
        append(h, base + rank, score_at(x), tok + x);
      }
      while (mask) {                                           // a second candidate in one group of eight: rare
        const uint32_t x = (uint32_t)__ffs((int)mask) - 1u;
        mask &= mask - 1u;
        append(h, atomicAdd(&M.ccount[h], 1u), score_at(x), tok + x);
      }
    }
    parked = 0u;
    __syncwarp();                                              // the ring may be written again
  };

  while (true) {
    // ---- the stage after this one: the next pass of the sub-tile, the next sub-tile of the tile, or my next tile
    int g_next = g, u_next = u, pass_next = pass + 1;
    if (pass_next == npass) {
      pass_next = 0;
      u_next = u + 1;
      if (u_next * tb >= TILE_BLOCKS || first_block(g) + u_next * tb >= nb_item) { u_next = 0; g_next = g + gridDim.x; }
    }
    const bool more = g_next < total;
    const bool same_item = more && g_next < B.tile_end[item];
    fathom_copies_wait<0>();
    __syncthreads();                                           // this stage's words and scales are in place, and every warp has
                                                               // left the previous stage: its buffer may be refilled
    if (same_item) prefetch(g_next, u_next, pass_next, buf ^ 1);   // lands while this stage is scanned

    // ---- eight consecutive scores of head t4 (lanes with t4 < NH, tokens of an existing block): tokens tok .. tok + 7 of
    //      the session, written at position dst of the head's row (MODE 0, 1) or tested against the head's threshold (MODE 2)
    auto emit = [&](const float (&v)[8], uint32_t tok, uint32_t dst, uint32_t n, bool live) {
      if (MODE != 2) {
        if (!live) return;
        float* row = B.scores[item] + (size_t)(h0 + t4) * (size_t)B.score_stride[item] + dst;
        if (tok + 8 <= n) {
          store_scores8(row, v);
        } else {
#pragma unroll
          for (int x = 0; x < 8; ++x)
            if (tok + x < n) row[x] = v[x];
        }
      } else {
        // a lane with a candidate among its eight scores parks them (called by all lanes of the warp; `live`: the lane
        // has scores at all).  Eligibility of the tokens is checked when the ring is sifted.
        const float vmax = fmaxf(fmaxf(fmaxf(v[0], v[1]), fmaxf(v[2], v[3])), fmaxf(fmaxf(v[4], v[5]), fmaxf(v[6], v[7])));
        const bool has = live && vmax >= my_thr;
        const unsigned bal = __ballot_sync(0xffffffffu, has);
        if (bal) {                                             // (the same for every lane)
          if (has) {
            const uint32_t e = warp * PARK_RING + parked + __popc(bal & ((1u << lane) - 1u));
            M.park_lo[e] = make_float4(v[0], v[1], v[2], v[3]);
            M.park_hi[e] = make_float4(v[4], v[5], v[6], v[7]);
            M.park_tok[e] = tok | ((uint32_t)t4 << 30);
          }
          parked += __popc(bal);
          if (parked > (uint32_t)(PARK_RING - 32)) sift();
        }
      }
    };

    // ---- a whole stage of TB blocks and NKS x 16 rows, single pass: the warp's TB / 4 blocks are 16 TB tokens, and a lane
    //      takes 2 TB consecutive ones (TB = 16: half a block, TB = 8: a quarter): ONE load of TB / 4 bytes per row gives all
    //      their bits, and one scale pair per row pair serves them all.  They are worked eight at a time (byte k of the
    //      loaded words): slice j of the accumulators then holds tokens 8 k + 2 j (mma row gq) and 8 k + 2 j + 1 (row gq + 8)
    //      of the lane's tokens
    auto owned_tokens = [&](auto tbc, auto nksc, int blk0) {
      constexpr int TB = decltype(tbc)::value, NKS = decltype(nksc)::value;
      constexpr int BYTES = TB / 4;                            // plane bytes per row and lane
      using GE = Geo<TB>;
      const int mine = warp * (TB / 4) + (gq * BYTES) / 8;     // my block of the stage
      const int off = (gq * BYTES) % 8;                        // where my bytes start in its words
      const unsigned char* wp = M.words[buf] + (2 * t4) * GE::ROW_BYTES + mine * 8 + off;
      const uint16_t* sp = reinterpret_cast<const uint16_t*>(M.scale[buf]) + (2 * t4) * GE::SCALE_ELEMS + mine;
      uint32_t w[NKS][4], S[NKS][2];
      uint2 bf[NKS];
      auto plane_bytes = [](const unsigned char* p) -> uint32_t {
        return BYTES == 4 ? *reinterpret_cast<const uint32_t*>(p) : (uint32_t)*reinterpret_cast<const uint16_t*>(p);
      };
#pragma unroll
      for (int ks = 0; ks < NKS; ++ks) {
        bf[ks] = M.bfr[ks][lane];
        const unsigned char* wk = wp + ks * (16 * GE::ROW_BYTES);
        w[ks][0] = plane_bytes(wk);
        w[ks][1] = plane_bytes(wk + GE::ROW_BYTES);
        w[ks][2] = plane_bytes(wk + 8 * GE::ROW_BYTES);
        w[ks][3] = plane_bytes(wk + 9 * GE::ROW_BYTES);
        const uint16_t* sk = sp + ks * (16 * GE::SCALE_ELEMS);
        S[ks][0] = __byte_perm(sk[0], sk[GE::SCALE_ELEMS], 0x5410);
        S[ks][1] = __byte_perm(sk[8 * GE::SCALE_ELEMS], sk[9 * GE::SCALE_ELEMS], 0x5410);
      }
      const uint32_t n = (uint32_t)B.n[item];
      const uint32_t tok0 = (uint32_t)(blk0 + mine) * FATHOM_BLOCK + off * 8;            // my first token
      const uint32_t dst0 = MODE == 1 ? (uint32_t)g * (TILE_BLOCKS * FATHOM_BLOCK) + (uint32_t)(u * TB + mine) * FATHOM_BLOCK + off * 8 : tok0;
#pragma unroll
      for (int k = 0; k < BYTES; ++k) {
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
#pragma unroll
        for (int ks = 0; ks < NKS; ++ks) {
          // byte k of the two rows of a pair side by side: bits 0..7 and 16..23 (the other bytes are masked away later)
          const uint32_t x0 = __byte_perm(w[ks][0], w[ks][1], 0x0400 + 0x0101 * k);
          const uint32_t x1 = __byte_perm(w[ks][2], w[ks][3], 0x0400 + 0x0101 * k);
          const uint32_t S0 = S[ks][0], S1 = S[ks][1];
          mma_16816(acc[0], signed_pair<15>(S0, x0), signed_pair<14>(S0, x0), signed_pair<15>(S1, x1), signed_pair<14>(S1, x1), bf[ks].x, bf[ks].y);
          mma_16816(acc[1], signed_pair<13>(S0, x0), signed_pair<12>(S0, x0), signed_pair<13>(S1, x1), signed_pair<12>(S1, x1), bf[ks].x, bf[ks].y);
          mma_16816(acc[2], signed_pair<11>(S0, x0), signed_pair<10>(S0, x0), signed_pair<11>(S1, x1), signed_pair<10>(S1, x1), bf[ks].x, bf[ks].y);
          mma_16816(acc[3], signed_pair<9>(S0, x0), signed_pair<8>(S0, x0), signed_pair<9>(S1, x1), signed_pair<8>(S1, x1), bf[ks].x, bf[ks].y);
        }
        float v[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[2 * j] = fmaf(acc[j][1], hs_tail, acc[j][0] * hs);
          v[2 * j + 1] = fmaf(acc[j][3], hs_tail, acc[j][2] * hs);
        }
        emit(v, tok0 + 8 * k, dst0 + 8 * k, n, t4 < NH);
      }
    };

    auto compute = [&](auto tbc) {
      constexpr int TB = decltype(tbc)::value;
      using GE = Geo<TB>;
      constexpr int BW = TB / WARPS;                           // blocks per warp and stage
      const int s0 = pass * GE::ROWS, sc = min(GE::ROWS, nrows - s0), nks = (sc + 15) >> 4;
      const int blk0 = first_block(g) + u * TB;
      const uint32_t n = (uint32_t)B.n[item];                  // n < 2^31
      if constexpr (TB >= 8) if (npass == 1 && nks >= 1 && (uint32_t)(blk0 + TB) * FATHOM_BLOCK <= n) {
        // ---- the common stages (plans of up to 96 rows, whole sub-tiles of a long sequence)
        constexpr int K0 = TB == 16 ? 0 : 3;                   // TB = 8 serves 49 .. 96 rows: 4 .. 6 steps of 16
        if (nks == K0 + 3) owned_tokens(tbc, std::integral_constant<int, K0 + 3>(), blk0);
        else if (nks == K0 + 2) owned_tokens(tbc, std::integral_constant<int, K0 + 2>(), blk0);
        else owned_tokens(tbc, std::integral_constant<int, K0 + 1>(), blk0);
        return;
      }
#pragma unroll 1
      for (int i = 0; i < BW; ++i) {
        const int b = warp * BW + i;                           // my block within the sub-tile
        if (pass == 0) {
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.0f;
        }
        // my byte (tokens 8 gq .. 8 gq + 7) of the plane words and the scales of rows 2 t4, 2 t4 + 1 (+ 8, + 9) of every 16
        const unsigned char* wp = M.words[buf] + (2 * t4) * GE::ROW_BYTES + b * 8 + gq;
        const uint16_t* sp = reinterpret_cast<const uint16_t*>(M.scale[buf]) + (2 * t4) * GE::SCALE_ELEMS + b;
        const uint2* bfr_lane = &M.bfr[0][lane];
        if (nks == 3) mma_rows<GE::ROW_BYTES, GE::SCALE_ELEMS, 3>(acc, wp, sp, bfr_lane, 3);   // 33 .. 48 rows: a B = 48 plan
        else mma_rows<GE::ROW_BYTES, GE::SCALE_ELEMS, 0>(acc, wp, sp, bfr_lane, nks);
        if (pass != npass - 1) continue;

        // ---- scores of head t4 for my eight tokens: columns 2 t4 (head part) and 2 t4 + 1 (tail part)
        float v[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          v[2 * j] = fmaf(acc[j][1], hs_tail, acc[j][0] * hs);
          v[2 * j + 1] = fmaf(acc[j][3], hs_tail, acc[j][2] * hs);
        }
        const bool have_block = blk0 + b < nb_item;
        const uint32_t tok = (uint32_t)(blk0 + b) * FATHOM_BLOCK + gq * 8;                     // my first token
        emit(v, tok, MODE == 1 ? (uint32_t)g * (TILE_BLOCKS * FATHOM_BLOCK) + (uint32_t)(u * TB + b) * FATHOM_BLOCK + gq * 8 : tok, n,
             t4 < NH && have_block);
      }
    };
    if (tb == 16) compute(std::integral_constant<int, 16>());
    else if (tb == 8) compute(std::integral_constant<int, 8>());
    else compute(std::integral_constant<int, 4>());

    if (MODE == 2 && (++stages & 3u) == 0u) sift();            // (every warp of the CTA at the same stages)
    if (!more) break;
    g = g_next;
    u = u_next;
    pass = pass_next;
    buf ^= 1;
    if (!same_item) {                                          // first tile of another session: nothing was fetched ahead
      __syncthreads();                                         // every warp is done with the previous session's row list
      enter_item(g);
      prefetch(g, 0, 0, buf);
      fill_bfr(0);
    } else if (npass > 1) {
      __syncthreads();                                         // every warp is done with the previous pass's right operand
      fill_bfr(pass);                                          // plans of more than 160 rows: the right operand of the next pass
    }
  }
  if (MODE == 2) {
    // ---- the CTA has scanned its last tile: what is still parked is sifted, then the four lists go to the heads' global
    //      lists, one atomic per head
    sift();
    __syncthreads();
    if (tid < NH) {
      const uint32_t c = min(M.ccount[tid], (uint32_t)CAND_LIST);
      M.ccount[tid] = c;
      M.cbase[tid] = c ? atomicAdd(&fz.cand_count[h0 + tid], c) : 0u;
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < NH && h < 4; ++h) {
      const uint32_t c = M.ccount[h], at = M.cbase[h];
      for (uint32_t e = tid; e < c; e += THREADS)
        if ((long long)(at + e) < fz.capacity) {
          const uint2 it = M.clist[h * CAND_LIST + e];
          fz.cand_score[(size_t)(h0 + h) * fz.capacity + at + e] = __uint_as_float(it.x);
          fz.cand_idx[(size_t)(h0 + h) * fz.capacity + at + e] = (int32_t)it.y;
        }
    }
  }
}

template <int NH, int MODE>
int launch_scan(const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz, bool dependent,
                cudaStream_t st) {
  const long long tiles = B.tile_end[B.items - 1];
  if (tiles <= 0) return FATHOM_OK;
  const int plans = Hq / NH;
  bool host = false;                                          // any store of the launch in pinned host memory
  for (int i = 0; i < B.items; ++i) host = host || fathom_planes_in_host_memory(B.planes[i]);
  dim3 grid((unsigned)fathom_scan_grid_ctas(tiles, plans, host, CTAS_PER_SM), (unsigned)plans);
  constexpr size_t smem = sizeof(Smem<MODE>);                 // dynamic: MODE 2 needs more than the static limit
  auto kernel = host ? scan_kernel<NH, MODE, false> : scan_kernel<NH, MODE, true>;
  if (smem > 48 * 1024) {
    static bool configured[64][2] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return FATHOM_ERR_CUDA;
    if (dev >= 0 && dev < 64 && !configured[dev][host ? 0 : 1]) {
      if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) return FATHOM_ERR_CUDA;
      configured[dev][host ? 0 : 1] = true;
    }
  }
  if (dependent) {                                            // may become resident while the previous kernel of the stream runs
    if (fathom_launch_dependent(kernel, grid, dim3(THREADS), smem, st, B, Hq / Hkv, heads_per_plan, fz) != cudaSuccess)
      return FATHOM_ERR_CUDA;
    return FATHOM_OK;
  }
  kernel<<<grid, THREADS, smem, st>>>(B, Hq / Hkv, heads_per_plan, fz);
  return FATHOM_OK;
}

// FATHOM_SCAN_PATH=simt (read once) selects the CUDA-core kernel of scan_simt.cu for every scan of the process
bool simt_path() {
  static const bool v = [] { const char* e = getenv("FATHOM_SCAN_PATH"); return e && strcmp(e, "simt") == 0; }();
  return v;
}

template <int MODE>
int dispatch_scan(const ScanBatch& B, int Hkv, int Hq, int heads_per_plan, const fathom_scan_fuse& fz, bool dependent,
                  cudaStream_t st) {
  if (simt_path()) return fathom_scan_simt_dispatch(MODE, B, Hkv, Hq, heads_per_plan, fz, dependent, st);
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

int g_ctas_override = 0;                                       // fathom_scan_set_ctas_per_plan

}  // namespace

// Whether the planes are read over the host link (pinned host memory mapped into the device's address space)
bool fathom_planes_in_host_memory(const void* planes) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, planes) != cudaSuccess) { cudaGetLastError(); return false; }
  return a.type == cudaMemoryTypeHost;
}

int fathom_scan_ctas_override() { return g_ctas_override; }

int fathom_scan_grid_ctas(long long tiles, int plans, bool host_planes, int ctas_per_sm) {
  if (g_ctas_override >= 1) return (int)(g_ctas_override < tiles ? g_ctas_override : tiles);
  if (host_planes) return (int)tiles;
  static int sms[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  if (!sms[dev]) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0) v = 148;
    sms[dev] = v;
  }
  long long x = (long long)sms[dev] * ctas_per_sm / plans;
  if (x < 1) x = 1;
  return (int)(x < tiles ? x : tiles);
}

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
  // (a programmatic dependent: the second, gated attempt then costs no launch latency when it has nothing to do)
  if (L->n > (1ll << 30)) return FATHOM_ERR_UNSUPPORTED;      // a parked group keeps its first token in 30 bits
  return dispatch_scan<2>(single_item(L, planes, scales, q, depth, nullptr, 0, 1), L->n_kv_heads, L->n_q_heads, heads_per_plan, fz,
                          true, st);
}

extern "C" int fathom_scan_set_ctas_per_plan(int ctas) {
  g_ctas_override = ctas > 0 ? ctas : 0;
  return FATHOM_OK;
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
