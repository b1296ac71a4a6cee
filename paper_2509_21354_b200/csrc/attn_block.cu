// Host side of the block-of-queries attention (kvE_decode_attn_block): tensor maps over the page pools
// and the summary store, and the launch.  The kernel is in attn_block_tc.cu.
#include "attn_block.cuh"

namespace kve {

cudaError_t launch_attn_block_tc(const CUtensorMap* tm, const BlockArgs& a, dim3 grid, cudaStream_t st);

// ---- host side ------------------------------------------------------------------------------------
int attn_block_hp(int C) {
  int hp = 64;
  while (hp > 1 && C % hp != 0) hp >>= 1;
  return hp;
}

// [rows][128] bf16, boxes of 64 columns x box_rows rows, 128-byte swizzle
static cudaError_t encode_rows_map(CUtensorMap* tm, const void* base, unsigned long long rows, unsigned box_rows) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static EncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = reinterpret_cast<EncodeFn>(fn);
  }
  if (rows == 0 || rows >= (1ULL << 31)) return cudaErrorInvalidValue;
  const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ROW_BYTES};
  const cuuint32_t box[2] = {64u, box_rows};
  const cuuint32_t estr[2] = {1u, 1u};
  const CUresult r = encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

static_assert(sizeof(CUtensorMap) == ATTN_BLOCK_MAP_BYTES, "tensor map size");

cudaError_t encode_attn_block_maps(void* maps, const void* k_pages, const void* v_pages, long long page_rows, int hp,
                                   const void* ksum, const void* vsum, long long sum_rows) {
  CUtensorMap* tm = static_cast<CUtensorMap*>(maps);
  cudaError_t e = encode_rows_map(tm + 0, k_pages, (unsigned long long)page_rows, (unsigned)hp);
  if (e == cudaSuccess) e = encode_rows_map(tm + 1, v_pages, (unsigned long long)page_rows, (unsigned)hp);
  if (e == cudaSuccess) e = encode_rows_map(tm + 2, ksum, (unsigned long long)sum_rows, (unsigned)ATTN_BLOCK_SUM_BOX);
  if (e == cudaSuccess) e = encode_rows_map(tm + 3, vsum, (unsigned long long)sum_rows, (unsigned)ATTN_BLOCK_SUM_BOX);
  return e;
}

cudaError_t launch_attn_block(const LayerView& v, const void* maps, AttnMode mode, int n_chunks, AttnPlan plan, int T, int G,
                              int causal, int hp, long long sum_row0, const void* q, void* out, float* lse, float scale, float* partials,
                              int32_t* counters, cudaStream_t st) {
  if (v.S <= 0 || T <= 0) return cudaSuccess;
  const int R = T * G;
  if (R > ATTN_BLOCK_MAX_ROWS || hp < 8) return cudaErrorInvalidValue;
  BlockArgs a;
  a.v = v; a.mode = (int)mode; a.n_chunks = n_chunks;
  a.rows_per_split = plan.rows_per_split; a.max_splits = plan.max_splits;
  a.T = T; a.G = G; a.R = R; a.rec_rows = (R + 15) / 16 * 16; a.causal = causal; a.hp = hp; a.sum_row0 = sum_row0;
  a.q = static_cast<const uint16_t*>(q); a.out = static_cast<uint16_t*>(out); a.lse = lse; a.scale = scale;
  a.partials = partials; a.counters = counters;
  const CUtensorMap* tm = static_cast<const CUtensorMap*>(maps);
  dim3 grid((unsigned)plan.max_splits, (unsigned)v.S);
  return launch_attn_block_tc(tm, a, grid, st);
}

}  // namespace kve
