// CUDA-core expert FFN: one thread per weight row, pages read tile by tile with contiguous 16-byte
// loads, dequantized in registers, fp32 accumulation against up to eight tokens at a time.  An
// independent second implementation of the expert FFN (PW_MODE_SIMT): the tests run it beside the
// tensor-core kernels.  It is far slower than those at every batch size, so PW_MODE_AUTO never picks it.
#include "pw_common.cuh"
#include "pw_layout.cuh"

namespace pw {

constexpr int kSimtTok = 8;  // tokens per pass over the weights

template <int BITS>
__device__ __forceinline__ void load_decode_group(const DevRow& row, size_t tile, int r, __half2* w) {
  const char* tile_base = reinterpret_cast<const char*>(row.codes) + tile * tile_bytes(BITS);
  const uint4* tb = reinterpret_cast<const uint4*>(tile_base) + r;
  __half2 s2 = __half2half2(__ushort_as_half((unsigned short)0x3c00)), z2 = s2;
  if constexpr (BITS < 16) {
    s2 = __half2half2(*reinterpret_cast<const __half*>(tile_base + tile_scale_offset(BITS, r)));
    z2 = __half2half2(*reinterpret_cast<const __half*>(tile_base + tile_zp_offset(BITS, r)));
  }
  decode_half<BITS>(tb, 0, s2, z2, w);
  decode_half<BITS>(tb, 1, s2, z2, w + 32);
}

__device__ __forceinline__ void decode_any(const DevRow& row, size_t tile, int r, __half2* w) {
  switch (row.bits) {
    case 16: load_decode_group<16>(row, tile, r, w); break;
    case 8: load_decode_group<8>(row, tile, r, w); break;
    case 4: load_decode_group<4>(row, tile, r, w); break;
    case 3: load_decode_group<3>(row, tile, r, w); break;
    default: load_decode_group<2>(row, tile, r, w); break;
  }
}

__device__ __forceinline__ void fma_group(const __half2* w, const uint4 (*xs)[kSimtTok], float* acc) {
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    float2 wf[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) wf[i] = __half22float2(w[4 * c + i]);
#pragma unroll
    for (int n = 0; n < kSimtTok; ++n) {
      const uint4 xv = xs[c][n];
      const __half2* xh = reinterpret_cast<const __half2*>(&xv);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 xf = __half22float2(xh[i]);
        acc[n] = fmaf(wf[i].x, xf.x, acc[n]);
        acc[n] = fmaf(wf[i].y, xf.y, acc[n]);
      }
    }
  }
}

// PHASE 0: h = silu(W_gate x) * (W_up x) -> Ht (fp16, k-chunk major).  PHASE 1: y = W_down h -> Y.
template <int PHASE>
__global__ void __launch_bounds__(128) ffn_simt_kernel(const DevRow* __restrict__ rows, const int32_t* __restrict__ offsets,
                                                       const uint4* __restrict__ bop, int Rpad, __half* __restrict__ ht,
                                                       float* __restrict__ y, int H) {
  __shared__ uint4 xs[16][kSimtTok];
  const int seg = blockIdx.y, rt = blockIdx.x, r = threadIdx.x;
  const int n0 = offsets[seg], n1 = offsets[seg + 1];
  if (n0 == n1) return;
  const DevRow ra = rows[seg * 3 + (PHASE == 0 ? 0 : 2)];
  const DevRow rb = rows[seg * 3 + 1];
  const int ng = ra.cols / kGroup;
  for (int nb = n0; nb < n1; nb += kSimtTok) {
    float acc_a[kSimtTok], acc_b[kSimtTok];
#pragma unroll
    for (int n = 0; n < kSimtTok; ++n) acc_a[n] = acc_b[n] = 0.f;
    for (int g = 0; g < ng; ++g) {
      __syncthreads();
      {
        const int c = r >> 3, n = r & 7;
        xs[c][n] = bop[(size_t)(g * 16 + c) * Rpad + nb + n];
      }
      __syncthreads();
      const size_t tile = (size_t)rt * ng + g;
      __half2 w[64];
      decode_any(ra, tile, r, w);
      fma_group(w, xs, acc_a);
      if (PHASE == 0) {
        decode_any(rb, tile, r, w);
        fma_group(w, xs, acc_b);
      }
    }
    const int row = rt * kTileRows + r;
#pragma unroll
    for (int n = 0; n < kSimtTok; ++n) {
      if (nb + n >= n1) break;
      if (PHASE == 0) {
        const float gte = acc_a[n];
        const float h = __fmul_rn(__fdiv_rn(gte, __fadd_rn(1.0f, expf(-gte))), acc_b[n]);
        ht[((size_t)(row >> 3) * Rpad + nb + n) * 8 + (row & 7)] = __float2half_rn(h);
      } else {
        y[(size_t)(nb + n) * H + row] = acc_a[n];
      }
    }
  }
}

pw_status launch_ffn_simt(pw_ctx* ctx, int layer, int T, int k, cudaStream_t s) {
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  char* b = ctx->base;
  const DevRow* rows = reinterpret_cast<const DevRow*>(b + w.table) + (size_t)layer * w.S * 3;
  const int32_t* offsets = reinterpret_cast<const int32_t*>(b + w.offsets);
  timing_mark(ctx, PW_K_FFN_GATE_UP, s);
  ffn_simt_kernel<0><<<dim3(c.ffn / kTileRows, w.S), 128, 0, s>>>(rows, offsets, reinterpret_cast<const uint4*>(b + w.xt),
                                                                  w.Rpad, reinterpret_cast<__half*>(b + w.ht), nullptr,
                                                                  c.hidden);
  timing_mark(ctx, PW_K_FFN_DOWN, s);
  ffn_simt_kernel<1><<<dim3(c.hidden / kTileRows, w.S), 128, 0, s>>>(rows, offsets,
                                                                     reinterpret_cast<const uint4*>(b + w.ht), w.Rpad,
                                                                     nullptr, reinterpret_cast<float*>(b + w.y),
                                                                     c.hidden);
  ctx->launches += 2;
  PW_CUDA_OK(cudaGetLastError());
  (void)T;
  (void)k;
  return PW_OK;
}

}  // namespace pw
