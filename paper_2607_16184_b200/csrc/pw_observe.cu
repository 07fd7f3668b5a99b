// Observation taps of a layer call: the sums behind the routing mass of every expert (Eq. 1) and behind the
// routed-input features of every linear-block (Sec. 3.2: routing-weighted mean and RMS input norm, maximum
// input norm).  They are by-products of buffers the forward call has just filled -- the gathered token rows,
// the SwiGLU rows, the gates and the grouping -- so one small kernel at the end of the call's chain reads
// them while they are still in L2.  All sums are taken in a fixed order: the same calls give the same bits.
#include "pw_common.cuh"

namespace pw {

// part[(z * 2 + which) * Rpad + n] = sum of squares of slice z of operand row n; which = 0: token rows
// ([H/8][Rpad][8] fp16), which = 1: SwiGLU rows ([F/8][Rpad][8] fp16).  A CTA takes 32 rows; its eight warps
// stride over the slice's k-chunks, so every load instruction of a warp reads 512 contiguous bytes.
__device__ __forceinline__ float warp_sum(float v);
__device__ __forceinline__ float warp_max(float v);
__device__ void accumulate_segment(const float* part, int Rpad, const int32_t* __restrict__ offsets,
                                   const int32_t* __restrict__ perm, const float* __restrict__ gates, int E, int s,
                                   int lane, float* __restrict__ acc);

__global__ void __launch_bounds__(256) row_norm_kernel(const uint4* __restrict__ xt, int chunks_x,
                                                       const uint4* __restrict__ ht, int chunks_h, int Rpad, int R,
                                                       float* part, int32_t* __restrict__ done_counter,
                                                       const int32_t* __restrict__ offsets,
                                                       const int32_t* __restrict__ perm,
                                                       const float* __restrict__ gates, int E, int S,
                                                       float* __restrict__ acc) {
  grid_dep_sync();
  grid_dep_trigger();
  __shared__ float sm[8][32];
  __shared__ int is_last;
  const int which = blockIdx.y, z = blockIdx.z;
  const uint4* buf = which ? ht : xt;
  const int chunks = which ? chunks_h : chunks_x;
  const int c0 = (int)(((long long)chunks * z) / kNormSplit), c1 = (int)(((long long)chunks * (z + 1)) / kNormSplit);
  const int r = threadIdx.x & 31, cl = threadIdx.x >> 5;
  const int n = blockIdx.x * 32 + r;
  float a = 0.f;
  if (n < R) {
#pragma unroll 8
    for (int c = c0 + cl; c < c1; c += 8) {        // independent loads: the unrolled loop keeps eight in flight
      const uint4 v = buf[(size_t)c * Rpad + n];
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
        a = fmaf(f.x, f.x, a);
        a = fmaf(f.y, f.y, a);
      }
    }
  }
  sm[cl][r] = a;
  __syncthreads();
  if (cl == 0 && n < R) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += sm[i][r];
    part[(size_t)(z * 2 + which) * Rpad + n] = s;
  }
  // The CTA that finishes last adds the call to the accumulators (a warp per segment, fixed order): one
  // launch instead of two, and still a single writer per accumulator row.
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) {
    const int total = (int)(gridDim.x * gridDim.y * gridDim.z);
    is_last = atomicAdd(done_counter, 1) == total - 1;
  }
  __syncthreads();
  if (!is_last) return;
  __threadfence();
  for (int s = cl; s < S; s += 8) accumulate_segment(part, Rpad, offsets, perm, gates, E, s, r, acc);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// One warp per expert segment: adds this call's pairs to the segment's eight accumulators (PW_OBS_*).  The
// routing weight of operand row n of a routed expert is the gate of the pair perm[n]; a shared expert takes
// every token with weight 1.  (`part` was written by other CTAs of this launch: read it past the L1.)
__device__ void accumulate_segment(const float* part, int Rpad, const int32_t* __restrict__ offsets,
                                   const int32_t* __restrict__ perm, const float* __restrict__ gates, int E, int s,
                                   int lane, float* __restrict__ acc) {
  const int n0 = offsets[s], n1 = offsets[s + 1];
  if (n1 <= n0) return;
  float sr = 0.f, srx = 0.f, srx2 = 0.f, mx = 0.f, srh = 0.f, srh2 = 0.f, mh = 0.f;
  for (int n = n0 + lane; n < n1; n += 32) {
    const float r = s < E ? gates[perm[n]] : 1.0f;
    float x2 = 0.f, h2 = 0.f;
#pragma unroll
    for (int z = 0; z < kNormSplit; ++z) {
      x2 += __ldcg(part + (size_t)(z * 2 + 0) * Rpad + n);
      h2 += __ldcg(part + (size_t)(z * 2 + 1) * Rpad + n);
    }
    const float nx = sqrtf(x2), nh = sqrtf(h2);
    sr += r;
    srx = fmaf(r, nx, srx);
    srx2 = fmaf(r, x2, srx2);
    mx = fmaxf(mx, nx);
    srh = fmaf(r, nh, srh);
    srh2 = fmaf(r, h2, srh2);
    mh = fmaxf(mh, nh);
  }
  sr = warp_sum(sr);
  srx = warp_sum(srx);
  srx2 = warp_sum(srx2);
  srh = warp_sum(srh);
  srh2 = warp_sum(srh2);
  mx = warp_max(mx);
  mh = warp_max(mh);
  if (lane == 0) {
    float* a = acc + (size_t)s * PW_OBS_FIELDS;
    a[PW_OBS_SUM_R] += sr;
    a[PW_OBS_PAIRS] += (float)(n1 - n0);
    a[PW_OBS_SUM_R_NX] += srx;
    a[PW_OBS_SUM_R_NX2] += srx2;
    a[PW_OBS_MAX_NX] = fmaxf(a[PW_OBS_MAX_NX], mx);
    a[PW_OBS_SUM_R_NH] += srh;
    a[PW_OBS_SUM_R_NH2] += srh2;
    a[PW_OBS_MAX_NH] = fmaxf(a[PW_OBS_MAX_NH], mh);
  }
}

// mass[e] = sum_r[e] / sum over the routed experts (Eq. 1); phi[(s * 3 + kind) * 3 + {mean, RMS, max}].
__global__ void __launch_bounds__(256) observe_summary_kernel(const float* __restrict__ acc, int E, int S,
                                                              float* __restrict__ mass, float* __restrict__ phi) {
  __shared__ float total;
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int e = 0; e < E; ++e) t += acc[(size_t)e * PW_OBS_FIELDS + PW_OBS_SUM_R];
    total = t;
  }
  __syncthreads();
  for (int s = threadIdx.x; s < S; s += blockDim.x) {
    const float* a = acc + (size_t)s * PW_OBS_FIELDS;
    const float sr = a[PW_OBS_SUM_R];
    if (mass && s < E) mass[s] = total > 0.f ? sr / total : 0.f;
    if (phi) {
      float fx[3] = {0.f, 0.f, 0.f}, fh[3] = {0.f, 0.f, 0.f};
      if (sr > 0.f) {
        fx[0] = a[PW_OBS_SUM_R_NX] / sr;
        fx[1] = sqrtf(a[PW_OBS_SUM_R_NX2] / sr);
        fx[2] = a[PW_OBS_MAX_NX];
        fh[0] = a[PW_OBS_SUM_R_NH] / sr;
        fh[1] = sqrtf(a[PW_OBS_SUM_R_NH2] / sr);
        fh[2] = a[PW_OBS_MAX_NH];
      }
      for (int d = 0; d < 3; ++d) {
        phi[((size_t)s * 3 + PW_GATE) * 3 + d] = fx[d];
        phi[((size_t)s * 3 + PW_UP) * 3 + d] = fx[d];
        phi[((size_t)s * 3 + PW_DOWN) * 3 + d] = fh[d];
      }
    }
  }
}

// The tail of a forward call: the taps (when the context has accumulators) and the closing timing mark.
pw_status launch_observe(pw_ctx* ctx, int layer, int T, int k, cudaStream_t s) {
  timing_mark(ctx, PW_K_OBSERVE, s);
  if (ctx->obs_acc) {
    const pw_config& c = ctx->cfg;
    const WsMap& w = ctx->ws;
    char* b = ctx->base;
    const int R = T * k + c.n_shared * T;
    float* part = reinterpret_cast<float*>(b + w.obs_part);
    PW_CUDA_OK(launch_dependent(row_norm_kernel, dim3((R + 31) / 32, 2, kNormSplit), dim3(256), 0, s,
                                reinterpret_cast<const uint4*>(b + w.xt), c.hidden / 8,
                                reinterpret_cast<const uint4*>(b + w.ht), c.ffn / 8, w.Rpad, R, part,
                                reinterpret_cast<int32_t*>(b + w.counter) + 2,   // zeroed by the grouping kernel
                                reinterpret_cast<const int32_t*>(b + w.offsets),
                                reinterpret_cast<const int32_t*>(b + w.perm),
                                reinterpret_cast<const float*>(b + w.gates), c.n_experts, w.S,
                                ctx->obs_acc + (size_t)layer * w.S * PW_OBS_FIELDS));
    ctx->launches += 1;
    PW_CUDA_OK(cudaGetLastError());
  }
  timing_mark(ctx, PW_NUM_KERNELS, s);
  return PW_OK;
}

}  // namespace pw

using namespace pw;

extern "C" pw_status pw_observe(pw_ctx* ctx, float* accumulators, pw_stream stream) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(accumulators) & 15) return PW_ERR_ALIGN;
  if (accumulators)
    PW_CUDA_OK(cudaMemsetAsync(accumulators, 0,
                               sizeof(float) * PW_OBS_FIELDS * (size_t)ctx->cfg.n_layers * ctx->ws.S, stream));
  ctx->obs_acc = accumulators;
  return PW_OK;
}

extern "C" pw_status pw_observation_summary(pw_ctx* ctx, int layer, float* mass, float* phi, pw_stream stream) {
  if (!ctx || (!mass && !phi)) return PW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return PW_ERR_INVALID_ARG;
  if (!ctx->obs_acc) return PW_ERR_STATE;
  if ((reinterpret_cast<uintptr_t>(mass) | reinterpret_cast<uintptr_t>(phi)) & 15) return PW_ERR_ALIGN;
  observe_summary_kernel<<<1, 256, 0, stream>>>(ctx->obs_acc + (size_t)layer * ctx->ws.S * PW_OBS_FIELDS,
                                                ctx->cfg.n_experts, ctx->ws.S, mass, phi);
  ctx->launches += 1;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}
