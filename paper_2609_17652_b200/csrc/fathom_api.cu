// Context management, argument validation and error text of libfathom.
#include "fathom_common.cuh"

#include <new>

int fathom_check_layout(const fathom_layout* L) {
  if (!L) return FATHOM_ERR_INVALID_ARG;
  if (L->n_kv_heads < 1 || L->n_q_heads < 1 || L->n < 1) return FATHOM_ERR_INVALID_ARG;
  if (L->n_q_heads % L->n_kv_heads != 0) return FATHOM_ERR_INVALID_ARG;
  if (L->d != FATHOM_D) return FATHOM_ERR_UNSUPPORTED;
  if (L->n > (int64_t)0x7fffffc0) return FATHOM_ERR_UNSUPPORTED;   // token indices are int32
  const int64_t nb = fathom_nblocks(L->n);
  if (L->plane_stride_words < nb || L->scale_stride < nb || L->score_stride < L->n) return FATHOM_ERR_INVALID_ARG;
  if (L->plane_stride_words % 2 != 0 || L->scale_stride % 8 != 0 || L->score_stride % 4 != 0) return FATHOM_ERR_ALIGNMENT;
  if (L->plane_stride_words >= ((int64_t)1 << 24) || L->scale_stride > (int64_t)0xffffffff) return FATHOM_ERR_UNSUPPORTED;   // row offsets in 16-byte units fit 32 bits
  return FATHOM_OK;
}

fathom_topk_scratch fathom_carve_topk(void* base, int Hq, int64_t n, int k) {
  fathom_topk_scratch s;
  char* p = static_cast<char*>(base);
  size_t off = 0;
  s.hist = reinterpret_cast<uint32_t*>(p + off);    off += fathom_round_up((size_t)Hq * FATHOM_TOPK_BINS * 4, 256);
  s.state = reinterpret_cast<uint32_t*>(p + off);   off += fathom_round_up((size_t)Hq * 8 * 4, 256);
  s.cand_count = reinterpret_cast<uint32_t*>(p + off); off += fathom_round_up((size_t)Hq * 4, 256);
  s.cand_count2 = reinterpret_cast<uint32_t*>(p + off); off += fathom_round_up((size_t)Hq * 4, 256);
  s.bitmap_words = (long long)((n + 1023) / 1024) * 32;                    // whole 32-word groups
  s.bitmap = reinterpret_cast<uint32_t*>(p + off);  off += fathom_round_up((size_t)Hq * (size_t)s.bitmap_words * 4, 256);
  s.cand = reinterpret_cast<int32_t*>(p + off);     off += fathom_round_up((size_t)Hq * (size_t)n * 4, 256);
  s.tile_count = reinterpret_cast<uint32_t*>(p + off); off += fathom_round_up((size_t)Hq * (size_t)((n + 8191) / 8192) * 4, 256);
  s.cand_score = reinterpret_cast<float*>(p + off); off += fathom_round_up((size_t)Hq * (size_t)n * 4, 256);
  {
    const long long tile = fathom_scan_tile_tokens();
    const int step = fathom_fused_tile_step(n, k);
    const long long sampled = ((n + tile - 1) / tile + step - 1) / step;
    s.sample_stride = step == 1 ? (long long)((n + 3) / 4 * 4) : sampled * tile;
    s.sample = reinterpret_cast<float*>(p + off);   off += fathom_round_up((size_t)Hq * (size_t)s.sample_stride * 4, 256);
  }
  s.bytes = off;
  return s;
}

fathom_attn_scratch fathom_carve_attn(void* base, int Hq, int k) {
  fathom_attn_scratch s;
  s.splits = (k + FATHOM_ATTN_CHUNK - 1) / FATHOM_ATTN_CHUNK;
  s.partial = static_cast<float*>(base);
  s.bytes = fathom_round_up((size_t)Hq * s.splits * (FATHOM_D + 2) * sizeof(float), 256);
  return s;
}

extern "C" {

size_t fathom_scratch_bytes(const fathom_layout* L, int k) {
  if (fathom_check_layout(L) != FATHOM_OK || k < 1) return 0;
  size_t a = fathom_carve_topk(nullptr, L->n_q_heads, L->n, k).bytes;
  size_t b = fathom_carve_attn(nullptr, L->n_q_heads, k).bytes;
  size_t c = fathom_union_scratch_bytes(L->n_kv_heads, L->n, (L->n_q_heads / L->n_kv_heads) * k);
  size_t e = fathom_calib_scratch_bytes(L->n_kv_heads, L->n);
  size_t r = fathom_rotate_tc_scratch_bytes(L->n_kv_heads);
  if (r > e) e = r;
  size_t m = a > b ? a : b;
  m = m > c ? m : c;
  return m > e ? m : e;
}

int fathom_create(fathom_ctx** out, int device, size_t scratch_bytes) {
  if (!out) return FATHOM_ERR_INVALID_ARG;
  *out = nullptr;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return FATHOM_ERR_CUDA;
  if (cudaSetDevice(device) != cudaSuccess) return FATHOM_ERR_CUDA;
  fathom_ctx* c = new (std::nothrow) fathom_ctx();
  if (!c) { cudaSetDevice(prev); return FATHOM_ERR_INVALID_ARG; }
  c->device = device;
  c->scratch = nullptr;
  c->scratch_bytes = scratch_bytes;
  c->dev_status = nullptr;
  c->last_cuda = cudaSuccess;
  cudaError_t e = cudaMalloc(&c->dev_status, FATHOM_CTL_BYTES);
  if (e == cudaSuccess) e = cudaMemset(c->dev_status, 0, FATHOM_CTL_BYTES);
  if (e == cudaSuccess && scratch_bytes > 0) e = cudaMalloc(&c->scratch, scratch_bytes);
  if (e != cudaSuccess) {
    if (c->dev_status) cudaFree(c->dev_status);
    delete c;
    cudaSetDevice(prev);
    return FATHOM_ERR_CUDA;
  }
  cudaSetDevice(prev);
  *out = c;
  return FATHOM_OK;
}

int fathom_destroy(fathom_ctx* c) {
  if (!c) return FATHOM_OK;
  int prev = 0;
  cudaGetDevice(&prev);
  cudaSetDevice(c->device);
  if (c->scratch) cudaFree(c->scratch);
  if (c->dev_status) cudaFree(c->dev_status);
  cudaSetDevice(prev);
  delete c;
  return FATHOM_OK;
}

const char* fathom_strerror(int status) {
  switch (status) {
    case FATHOM_OK: return "ok";
    case FATHOM_ERR_INVALID_ARG: return "invalid argument (null pointer, size or range)";
    case FATHOM_ERR_UNSUPPORTED: return "unsupported configuration (d must be 128; heads_per_plan in {1,2,4,8}; known mode/dtype)";
    case FATHOM_ERR_ALIGNMENT: return "pointer or stride is not 16-byte aligned as the layout requires";
    case FATHOM_ERR_SCRATCH_TOO_SMALL: return "context scratch arena is smaller than fathom_scratch_bytes() for this call";
    case FATHOM_ERR_CUDA: return "a CUDA runtime call failed (see fathom_last_cuda_error)";
    case FATHOM_ERR_STATIC_LIMIT: return "problem exceeds the built-in scratch of the allocation-free entry point (n_q_heads * ceil(k / 128) > FATHOM_ATTEND_STATIC_MAX_CHUNKS)";
    default: return "unknown fathom status";
  }
}

const char* fathom_last_cuda_error(const fathom_ctx* c) {
  return cudaGetErrorString(c ? c->last_cuda : cudaSuccess);
}

int fathom_device_status(fathom_ctx* c, void* stream, uint32_t* status) {
  if (!c || !status) return FATHOM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  FATHOM_CUDA_TRY(c, cudaMemcpyAsync(status, c->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, st));
  FATHOM_CUDA_TRY(c, cudaMemsetAsync(c->dev_status, 0, sizeof(uint32_t), st));
  FATHOM_CUDA_TRY(c, cudaStreamSynchronize(st));
  return FATHOM_OK;
}

int fathom_version(void) { return 100; }

}  // extern "C"
