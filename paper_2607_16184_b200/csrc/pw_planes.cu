// Overlaid bit-plane pages (PW_LAYOUT_PLANES): the nested quantizer that builds the three plane buffers of a
// block, and the export of the block's view at 2, 3 or 4 bits to the canonical page layout.  Lowering or raising
// the precision of such a block needs no kernel at all: the caller publishes the same buffers with another
// bitwidth.  One CTA per (128-row, one-group) tile, four threads per row, each owning a 32-weight slice.
#include "pw_common.cuh"
#include "pw_layout.cuh"
#include "pw_quant_core.cuh"

namespace pw {

// word of plane bits of one 32-weight slice: pair P = weights (2P, 2P + 1) at bit plane_bit_pos(P) of the low and
// of the high half-word
__device__ __forceinline__ uint32_t plane_word(const int (&code)[32], int bit) {
  uint32_t v = 0;
#pragma unroll
  for (int m = 0; m < 16; ++m) {
    v |= (uint32_t)((code[2 * m] >> bit) & 1) << plane_bit_pos(m);
    v |= (uint32_t)((code[2 * m + 1] >> bit) & 1) << (16 + plane_bit_pos(m));
  }
  return v;
}

__global__ void __launch_bounds__(512, 3) quant_planes_kernel(const __half* __restrict__ w, uint32_t cols,
                                                              char* __restrict__ top, char* __restrict__ bit1,
                                                              char* __restrict__ bit0) {
  const int g = blockIdx.x, rt = blockIdx.y, ng = gridDim.x;
  const int r = threadIdx.x >> 2, q = threadIdx.x & 3;
  const size_t tile = (size_t)rt * ng + g;
  float v[32];
  __half2 h16[16];
  const uint4* p = reinterpret_cast<const uint4*>(w + ((size_t)rt * kTileRows + r) * cols + (size_t)g * kGroup + 32 * q);
  uint4 u[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) u[i] = __ldg(p + i);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __half2* h = reinterpret_cast<const __half2*>(&u[i]);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(h[j]);
      h16[4 * i + j] = h[j];
      v[8 * i + 2 * j] = f.x;
      v[8 * i + 2 * j + 1] = f.y;
    }
  }
  int code[32];
  __half s4;
  float lo;
  group_quantize<true>(v, h16, 15, code, s4, lo);     // the 4-bit master code

  char* tb = top + tile * kPlaneTopTile;
  int hi2[32];
#pragma unroll
  for (int i = 0; i < 32; ++i) hi2[i] = code[i] >> 2;
  uint32_t tw[2];
  pack_slice<2>(hi2, tw);
  *reinterpret_cast<uint2*>(tb + slice_word_offset<2>(r, q, 0)) = make_uint2(tw[0], tw[1]);
  reinterpret_cast<uint32_t*>(bit1 + tile * kPlaneBitTile + r * 16)[q] = plane_word(code, 1);
  reinterpret_cast<uint32_t*>(bit0 + tile * kPlaneBitTile + r * 16)[q] = plane_word(code, 0);
  if (q == 0) {
    // lookup-table state of every bitwidth: scale x 2^(4-q) (exact), zero-point moved to the middle of the
    // levels that a shorter code merges (fp32 product, fp32 sum, one rounding to fp16)
    const float s = __half2float(s4);
    const __half sq[3] = {__float2half_rn(__fmul_rn(s, 4.0f)), __float2half_rn(__fmul_rn(s, 2.0f)), s4};
    const __half zq[3] = {__float2half_rn(__fadd_rn(lo, __fmul_rn(s, 1.5f))), __float2half_rn(__fadd_rn(lo, __fmul_rn(s, 0.5f))),
                          __float2half_rn(lo)};
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      __half* lut = reinterpret_cast<__half*>(tb + plane_lut_offset(2 + i));
      lut[r] = sq[i];
      lut[128 + r] = zq[i];
    }
  }
}

// The block's view at Q bits -> CANONICAL page (bit stream of the codes c4 >> (4 - Q), scales, zero-points).
template <int Q>
__global__ void __launch_bounds__(512) export_planes_kernel(const char* __restrict__ top, const char* __restrict__ bit1,
                                                            const char* __restrict__ bit0, uint32_t cols,
                                                            char* __restrict__ can_codes, __half* __restrict__ can_scales,
                                                            __half* __restrict__ can_zps) {
  const int g = blockIdx.x, rt = blockIdx.y, ng = gridDim.x;
  const int r = threadIdx.x >> 2, q = threadIdx.x & 3;
  const size_t tile = (size_t)rt * ng + g;
  const size_t row = (size_t)rt * kTileRows + r;
  const char* tb = top + tile * kPlaneTopTile;
  uint32_t tw[3];
  tw[0] = *reinterpret_cast<const uint32_t*>(tb + slice_word_offset<2>(r, q, 0));
  tw[1] = *reinterpret_cast<const uint32_t*>(tb + slice_word_offset<2>(r, q, 1));
  tw[2] = 0;
  int code[32];
  unpack_slice<2>(tw, code);
  if constexpr (Q >= 3) {
    const uint32_t b = reinterpret_cast<const uint32_t*>(bit1 + tile * kPlaneBitTile + r * 16)[q];
#pragma unroll
    for (int m = 0; m < 16; ++m) {
      code[2 * m] = (code[2 * m] << 1) | ((b >> plane_bit_pos(m)) & 1);
      code[2 * m + 1] = (code[2 * m + 1] << 1) | ((b >> (16 + plane_bit_pos(m))) & 1);
    }
  }
  if constexpr (Q == 4) {
    const uint32_t b = reinterpret_cast<const uint32_t*>(bit0 + tile * kPlaneBitTile + r * 16)[q];
#pragma unroll
    for (int m = 0; m < 16; ++m) {
      code[2 * m] = (code[2 * m] << 1) | ((b >> plane_bit_pos(m)) & 1);
      code[2 * m + 1] = (code[2 * m + 1] << 1) | ((b >> (16 + plane_bit_pos(m))) & 1);
    }
  }
  const size_t elem = row * cols + (size_t)g * kGroup + 32 * q;
  uint32_t* cpos = reinterpret_cast<uint32_t*>(can_codes + elem * Q / 8);     // 32 codes = Q whole words
  unsigned long long acc = 0;
  int nb = 0, wi = 0;
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    acc |= (unsigned long long)code[i] << nb;
    nb += Q;
    if (nb >= 32) {
      cpos[wi++] = (uint32_t)acc;
      acc >>= 32;
      nb -= 32;
    }
  }
  if (q == 0) {
    const __half* lut = reinterpret_cast<const __half*>(tb + plane_lut_offset(Q));
    can_scales[row * ng + g] = lut[r];
    can_zps[row * ng + g] = lut[128 + r];
  }
}

static bool aligned16p(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace pw

using namespace pw;

extern "C" size_t pw_plane_bytes(uint32_t rows, uint32_t cols, size_t* top_bytes, size_t* bit_bytes) {
  if (rows == 0 || cols == 0 || rows % kTileRows != 0 || cols % kGroup != 0) return 0;
  const size_t tiles = (size_t)(rows / kTileRows) * (cols / kGroup);
  if (top_bytes) *top_bytes = tiles * kPlaneTopTile;
  if (bit_bytes) *bit_bytes = tiles * kPlaneBitTile;
  return tiles * (kPlaneTopTile + 2 * kPlaneBitTile);
}

extern "C" pw_status pw_quantize_planes(pw_ctx* ctx, const void* w, uint32_t rows, uint32_t cols, pw_page* dst,
                                        pw_stream stream) {
  if (!ctx || !w || !dst) return PW_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0 || rows % kTileRows != 0 || cols % kGroup != 0) return PW_ERR_SHAPE;
  if (!dst->codes || !dst->scales || !dst->zps) return PW_ERR_INVALID_ARG;
  if (!aligned16p(w) || !aligned16p(dst->codes) || !aligned16p(dst->scales) || !aligned16p(dst->zps)) return PW_ERR_ALIGN;
  dst->rows = rows;
  dst->cols = cols;
  dst->group = kGroup;
  dst->bits = 4;
  dst->layout = PW_LAYOUT_PLANES;
  dim3 grid(cols / kGroup, rows / kTileRows);
  quant_planes_kernel<<<grid, 512, 0, stream>>>(reinterpret_cast<const __half*>(w), cols, reinterpret_cast<char*>(dst->codes),
                                                reinterpret_cast<char*>(dst->scales), reinterpret_cast<char*>(dst->zps));
  ctx->launches++;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

extern "C" pw_status pw_export_planes(pw_ctx* ctx, const pw_page* src, pw_page* dst, pw_stream stream) {
  if (!ctx || !src || !dst) return PW_ERR_INVALID_ARG;
  if (src->layout != PW_LAYOUT_PLANES) return PW_ERR_STATE;
  const int q = src->bits;
  if (q < 2 || q > 4) return PW_ERR_BITS;
  if (src->rows == 0 || src->cols == 0 || src->rows % kTileRows != 0 || src->cols % kGroup != 0 || src->group != kGroup)
    return PW_ERR_SHAPE;
  if (!src->codes || (q >= 3 && !src->scales) || (q == 4 && !src->zps)) return PW_ERR_STATE;   // a plane it needs is detached
  if (!dst->codes || !dst->scales || !dst->zps) return PW_ERR_INVALID_ARG;
  if (!aligned16p(src->codes) || !aligned16p(src->scales) || !aligned16p(src->zps) || !aligned16p(dst->codes) ||
      !aligned16p(dst->scales) || !aligned16p(dst->zps))
    return PW_ERR_ALIGN;
  dst->rows = src->rows;
  dst->cols = src->cols;
  dst->group = kGroup;
  dst->bits = (uint8_t)q;
  dst->layout = PW_LAYOUT_CANONICAL;
  dim3 grid(src->cols / kGroup, src->rows / kTileRows);
  const char* t = reinterpret_cast<const char*>(src->codes);
  const char* b1 = reinterpret_cast<const char*>(src->scales);
  const char* b0 = reinterpret_cast<const char*>(src->zps);
  char* cc = reinterpret_cast<char*>(dst->codes);
  __half* cs = reinterpret_cast<__half*>(dst->scales);
  __half* cz = reinterpret_cast<__half*>(dst->zps);
  switch (q) {
    case 2: export_planes_kernel<2><<<grid, 512, 0, stream>>>(t, b1, b0, src->cols, cc, cs, cz); break;
    case 3: export_planes_kernel<3><<<grid, 512, 0, stream>>>(t, b1, b0, src->cols, cc, cs, cz); break;
    default: export_planes_kernel<4><<<grid, 512, 0, stream>>>(t, b1, b0, src->cols, cc, cs, cz); break;
  }
  ctx->launches++;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}
