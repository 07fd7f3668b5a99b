// Token router (top-k + renormalised softmax gates), stable grouping of (token, slot) pairs into
// per-expert segments, operand gather, work-unit lists, and the gate-weighted combine.
#include "pw_common.cuh"

namespace pw {

constexpr int kMaxExpertsPerLane = 8;  // E <= 256
constexpr int kFusedRouteWork = 256;   // (token, choice) pairs x 32-expert strides up to which the grouping kernel routes itself

// Routing of one token by one warp.  Slot j holds the j-th largest logit; equal logits: lower expert index first.
template <int NS>   // NS = 32-expert strides a lane holds (1, 2, 4 or 8): the loops below cost in proportion
__device__ __forceinline__ void route_token_n(const float* __restrict__ logits, int token, int E, int k,
                                              int32_t* __restrict__ topk_ids, float* __restrict__ gates, int lane) {
  const float* l = logits + (size_t)token * E;
  float v[NS];
#pragma unroll
  for (int i = 0; i < NS; ++i) {
    const int e = lane + 32 * i;
    v[i] = e < E ? l[e] : -INFINITY;
  }
  uint32_t taken = 0;
  float l0 = 0.f, S = 0.f, myp = 0.f;
  int myid = 0;
  for (int j = 0; j < k; ++j) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < NS; ++i) {
      const int e = lane + 32 * i;
      const bool ok = e < E && !((taken >> i) & 1u);
      if (ok && (v[i] > bv || (v[i] == bv && e < bi))) {
        bv = v[i];
        bi = e;
      }
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, d);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, d);
      if (ov > bv || (ov == bv && oi < bi)) {
        bv = ov;
        bi = oi;
      }
    }
    if ((bi & 31) == lane) taken |= 1u << (bi >> 5);
    if (j == 0) l0 = bv;
    const float p = expf(__fsub_rn(bv, l0));
    S = __fadd_rn(S, p);  // summed in slot order, identically on every lane
    if (lane == j) {
      myp = p;
      myid = bi;
    }
  }
  // k <= 32: lane j owns slot j
  if (lane < k) {
    topk_ids[(size_t)token * k + lane] = myid;
    gates[(size_t)token * k + lane] = __fdiv_rn(myp, S);
  }
}

__device__ __forceinline__ void route_token(const float* __restrict__ logits, int token, int E, int k,
                                            int32_t* __restrict__ topk_ids, float* __restrict__ gates, int lane) {
  if (E <= 32) route_token_n<1>(logits, token, E, k, topk_ids, gates, lane);
  else if (E <= 64) route_token_n<2>(logits, token, E, k, topk_ids, gates, lane);
  else if (E <= 128) route_token_n<4>(logits, token, E, k, topk_ids, gates, lane);
  else route_token_n<kMaxExpertsPerLane>(logits, token, E, k, topk_ids, gates, lane);
}

// One warp per token.
__global__ void __launch_bounds__(256) router_kernel(const float* __restrict__ logits, int T, int E, int k,
                                                     int32_t* __restrict__ topk_ids, float* __restrict__ gates) {
  grid_dep_sync();   // the gates of the call before this one may still be read by its combine kernel
  grid_dep_trigger();
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= T) return;
  route_token(logits, warp, E, k, topk_ids, gates, lane);
}


// out[i] = in[0] + .. + in[i - 1] for i = 0 .. n (n + 1 results), by one warp, 32 values per step.
__device__ __forceinline__ void warp_exclusive_scan(const int32_t* in, int32_t* out, int n, int lane) {
  int carry = 0;
  for (int base = 0; base < n; base += 32) {
    const int i = base + lane;
    const int x = i < n ? in[i] : 0;
    int incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    if (i < n) out[i] = carry + incl - x;
    carry += __shfl_sync(0xffffffffu, incl, 31);
  }
  if (lane == 0) out[n] = carry;
}

// Single CTA.  Stable counting sort of the P = T*k pairs by expert (positions come from ordered
// prefix counts, never from atomics), segment table including the shared experts, operand-row ->
// token map, and the unit lists of the tensor-core kernels.  With `logits` given the CTA routes the tokens
// itself first (a warp per token, 32 at a time): for a decode batch that is cheaper than a launch of its own.
__global__ void __launch_bounds__(1024) permute_kernel(const float* __restrict__ logits, float* __restrict__ gates,
                                                       int32_t* topk_ids, int T, int k, int E,
                                                       int n_shared, int32_t* __restrict__ counts,
                                                       int32_t* __restrict__ offsets, int32_t* __restrict__ perm,
                                                       int32_t* __restrict__ inv_perm,
                                                       int32_t* __restrict__ row_token, int32_t* __restrict__ counter,
                                                       const DevRow* __restrict__ rows, int H, int F, int nt_tile,
                                                       int ksplit, int2* __restrict__ tile_tab, int max_tiles,
                                                       int32_t* __restrict__ n_units,
                                                       int32_t* __restrict__ seg_order, int max_units,
                                                       int32_t* __restrict__ status) {
  grid_dep_sync();
  grid_dep_trigger();
  extern __shared__ int32_t sm[];
  const int S = E + n_shared;
  int32_t* cnt = sm;                 // [S]
  int32_t* off = cnt + S;            // [S + 1]
  int32_t* run = off + S + 1;        // [E]   pairs of expert e placed so far
  int32_t* wcnt = run + E;           // [32][E]
  int32_t* ubase = wcnt + 32 * E;    // [S + 1] unit prefix (gate/up), reused for down
  int32_t* order = ubase + S + 1;    // [S]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = T * k;
  if (logits) {
    for (int t = warp; t < T; t += (int)(blockDim.x >> 5)) route_token(logits, t, E, k, topk_ids, gates, lane);
    __syncthreads();                                 // the pairs below are read back from global memory
  }
  for (int e = tid; e < S; e += blockDim.x) cnt[e] = e < E ? 0 : T;
  for (int e = tid; e < E; e += blockDim.x) run[e] = 0;
  if (tid < 64) counter[tid] = 0;
  __syncthreads();
  for (int p = tid; p < P; p += blockDim.x) atomicAdd(&cnt[topk_ids[p]], 1);
  __syncthreads();
  if (warp == 0) warp_exclusive_scan(cnt, off, S, lane);
  __syncthreads();
  for (int e = tid; e < S; e += blockDim.x) counts[e] = cnt[e];
  for (int e = tid; e <= S; e += blockDim.x) offsets[e] = off[e];

  for (int base = 0; base < P; base += blockDim.x) {
    for (int i = tid; i < 32 * E; i += blockDim.x) wcnt[i] = 0;
    __syncthreads();
    const int p = base + tid;
    const int e = p < P ? topk_ids[p] : -1;
    const uint32_t same = __match_any_sync(0xffffffffu, e);
    const int rank = __popc(same & ((1u << lane) - 1u));
    if (e >= 0 && rank == 0) wcnt[warp * E + e] = __popc(same);
    __syncthreads();
    for (int x = tid; x < E; x += blockDim.x) {
      int a = run[x];
      for (int w = 0; w < 32; ++w) {
        const int c = wcnt[w * E + x];
        wcnt[w * E + x] = a;
        a += c;
      }
      run[x] = a;
    }
    __syncthreads();
    if (e >= 0) {
      const int pos = off[e] + wcnt[warp * E + e] + rank;
      perm[pos] = p;
      inv_perm[p] = pos;
      row_token[pos] = p / k;
    }
    __syncthreads();
  }
  const int R = off[S];
  for (int i = tid; i < n_shared * T; i += blockDim.x) row_token[P + i] = i % T;
  for (int i = tid; i < kPadRows; i += blockDim.x) row_token[R + i] = -1;

  if (nt_tile <= 0) return;  // SIMT path: no unit lists

  // Tables of the unit lists (the lists themselves are written by the gather kernel, which has the threads
  // for it).  The CTAs of the FFN kernels claim units in list order, so the lists are laid out for that: row
  // tile outermost, K split next, then every segment's token tiles (segments with the widest pages first).
  // Consecutive units therefore belong to different experts -- pages of different bitwidths are in flight
  // together -- and the tiles that share weights are adjacent.  Here: per list, the token tiles in that
  // order.  Rank segments by counting (S is small); the sort's scratch is free by now and holds the bits.
  int32_t* sbits = wcnt;                           // gate + up bits | down bits << 16
  __syncthreads();
  for (int s = tid; s < S; s += blockDim.x)
    sbits[s] = (int32_t)((rows[s * 3].bits + rows[s * 3 + 1].bits) | (rows[s * 3 + 2].bits << 16));
  for (int phase = 0; phase < 2; ++phase) {
    __syncthreads();
    for (int s = tid; s < S; s += blockDim.x) {
      const int sh = phase == 0 ? 0 : 16;
      const uint32_t mine = ((uint32_t)sbits[s] >> sh) & 0xffffu;
      int rk = 0;
      for (int o = 0; o < S; ++o) {
        const uint32_t other = ((uint32_t)sbits[o] >> sh) & 0xffffu;
        rk += (other > mine) || (other == mine && o < s);
      }
      order[rk] = s;
    }
    __syncthreads();
    const int row_tiles = (phase == 0 ? F : H) / kTileRows;
    const int splits = phase == 0 ? 1 : ksplit;
    // token tiles per segment in rank order (in parallel), then their prefix (one warp)
    for (int i = tid; i < S; i += blockDim.x) ubase[i + 1] = (cnt[order[i]] + nt_tile - 1) / nt_tile;
    __syncthreads();
    if (warp == 0) warp_exclusive_scan(ubase + 1, ubase, S, lane);   // in place: a value is read before its slot is written
    if (tid == 0) {
      const int a = ubase[S];
      const long long total = (long long)a * row_tiles * splits;
      const bool fits = total <= max_units && a <= max_tiles;
      n_units[phase] = fits ? (int)total : 0;
      n_units[2 + phase] = a;                      // token tiles of the list
      if (!fits) atomicMax(status, (int)PW_ERR_NOMEM);
    }
    __syncthreads();
    if (ubase[S] > max_tiles) continue;
    if (phase == 0)
      for (int i = tid; i < S; i += blockDim.x) seg_order[i] = order[i];
    int2* tab = tile_tab + (size_t)phase * max_tiles;
    for (int i = tid; i < S; i += blockDim.x)
      for (int j = ubase[i]; j < ubase[i + 1]; ++j) tab[j] = make_int2(order[i], j - ubase[i]);
  }
}

// Xt[c][n][0..7] = hidden[row_token[n]][8c .. 8c+7] for the operand rows n < R.  Rows past R only ever feed
// accumulator columns that nobody reads, so they keep whatever they hold.
// The same grid first writes the two unit lists from the tables of the permute kernel: unit u of a list is
// (row tile, K split) pair u / TT and token tile u mod TT.
constexpr int kGatherChunks = 4;
// row_token, offsets, counts, tile_tab and n_units are written by the kernel directly ahead, during this kernel's
// lifetime: no __restrict__ on them, so that their loads cannot become non-coherent ones.
__global__ void __launch_bounds__(256) gather_kernel(const uint4* __restrict__ hidden, const int32_t* row_token,
                                                     const int32_t* offsets, int S, int H8, int Rpad,
                                                     uint4* __restrict__ xt, const int32_t* counts,
                                                     const int2* tile_tab, int max_tiles,
                                                     const int32_t* n_units, int nt_tile, int ksplit,
                                                     int ng_gu, int ng_dn, int dn_token_tile_outer,
                                                     Unit* __restrict__ units_gu, Unit* __restrict__ units_dn,
                                                     int32_t* __restrict__ done) {
  grid_dep_sync();
  grid_dep_trigger();
  if (nt_tile > 0) {
    const int gt = (blockIdx.y * gridDim.x + blockIdx.x) * blockDim.x + threadIdx.x;
    const int n_threads = gridDim.x * gridDim.y * blockDim.x;
    // completion counters of the gate/up units, one per (first operand row of a token tile, K range of the down
    // projection): the down kernel starts a unit as soon as the rows it multiplies are there
    for (int i = gt; i < offsets[S] * ksplit; i += n_threads) done[i] = 0;
    for (int phase = 0; phase < 2; ++phase) {
      const int total = n_units[phase], TT = n_units[2 + phase];
      const int splits = phase == 0 ? 1 : ksplit;
      const int ng = phase == 0 ? ng_gu : ng_dn;
      const int2* tab = tile_tab + (size_t)phase * max_tiles;
      Unit* out = phase == 0 ? units_gu : units_dn;
      // Row tile outermost by default: weight pages stream once, the token rows they multiply stay in L2.  When
      // the operand rows of the down projection do not fit in L2 (a long prompt: 235 MB at 4096 tokens of a
      // 14336-wide FFN) every row tile would pull them from HBM again; that list is laid out token tile
      // outermost instead -- a token tile's rows are read once, and the pages of its expert (the tables keep an
      // expert's token tiles together) are what stays in L2.
      const bool tt_outer = phase == 1 && dn_token_tile_outer;
      const int RS = TT > 0 ? total / TT : 0;
      for (int u = gt; u < total; u += n_threads) {
        int rs, j;
        if (tt_outer) {
          j = u / RS;
          rs = u - j * RS;
        } else {
          rs = u / TT;
          j = u - rs * TT;
        }
        // down projection: K range outermost, so that the units whose SwiGLU rows are finished first (the gate/up
        // list goes through the FFN rows in order) come first
        const int RT = RS / splits;
        const int sp = phase == 1 && !tt_outer ? rs / RT : rs % splits;
        const int rt = phase == 1 && !tt_outer ? rs - sp * RT : rs / splits;
        const int2 t = tab[j];
        const int n = counts[t.x];
        Unit un;
        un.seg = t.x;
        un.row_tile = rt;
        un.tok0 = offsets[t.x] + t.y * nt_tile;
        un.ntok = min(nt_tile, n - t.y * nt_tile);
        un.g0 = (sp * ng) / splits;
        un.g1 = ((sp + 1) * ng) / splits;
        un.split = sp;
        un.pad_ = 0;
        out[u] = un;
      }
    }
  }
  // kGatherChunks consecutive 16-byte chunks of one operand row per thread: the loads of a thread are in flight
  // together (64 contiguous bytes of the token's row), the stores of a warp are contiguous per chunk
  const int n = blockIdx.x * blockDim.x + threadIdx.x;
  const int c0 = blockIdx.y * kGatherChunks;
  if (n >= offsets[S]) return;
  const int t = row_token[n];
  uint4 v[kGatherChunks];
#pragma unroll
  for (int i = 0; i < kGatherChunks; ++i) {
    v[i] = make_uint4(0, 0, 0, 0);
    if (t >= 0 && c0 + i < H8) v[i] = __ldg(hidden + (size_t)t * H8 + c0 + i);
  }
#pragma unroll
  for (int i = 0; i < kGatherChunks; ++i)
    if (c0 + i < H8) xt[(size_t)(c0 + i) * Rpad + n] = v[i];
}

// out[t] = sum_j gate[t,j] * (sum_s y[s][inv_perm[t*k+j]]) + sum over shared experts (sum_s y[s][row]).
// A CTA takes 64 float4 columns of one token; its four thread rows each form the term of one expert choice at
// a time (all split-K partials are loaded before they are added, in split order), and thread row 0 adds the
// terms in choice order: the arithmetic and its order do not depend on the launch shape, only the latency does
// (a one-token call has a handful of CTAs, so a serial walk over choices x splits would be all latency).
constexpr int kCombineCols = 64, kCombineRows = 4, kMaxSplit = 8;
// kCombineChunks columns per thread, 64 apart: that many independent load chains in flight.  Four for a long
// prompt (thousands of tokens: fewer, fatter CTAs), one for a decode batch (more CTAs for the few tokens).
template <int kCombineChunks>
__global__ void __launch_bounds__(kCombineCols * kCombineRows)
    combine_kernel(const float4* y /* written by the kernel directly ahead */, const float* __restrict__ gates, const int32_t* __restrict__ inv_perm,
                   int T, int k, int n_shared, int H4, int ksplit, size_t split_stride4, float4* __restrict__ out) {
  grid_dep_sync();
  grid_dep_trigger();
  __shared__ float4 term[kCombineRows][kCombineChunks][kCombineCols];
  const int tx = threadIdx.x, ty = threadIdx.y;
  const int c_first = blockIdx.x * (kCombineCols * kCombineChunks) + tx;
  const int t = blockIdx.y;
  const int J = k + n_shared;
  float4 acc[kCombineChunks];
#pragma unroll
  for (int cc = 0; cc < kCombineChunks; ++cc) acc[cc] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < J; j0 += kCombineRows) {
    const int j = j0 + ty;
    if (j < J) {
      int row;
      float g;
      if (j < k) {
        row = inv_perm[(size_t)t * k + j];
        g = gates[(size_t)t * k + j];
      } else {
        row = T * k + (j - k) * T + t;
        g = 1.0f;
      }
#pragma unroll
      for (int cc = 0; cc < kCombineChunks; ++cc) {
        const int c = c_first + cc * kCombineCols;
        if (c >= H4) continue;
        float4 v[kMaxSplit];
#pragma unroll
        for (int s = 0; s < kMaxSplit; ++s)
          if (s < ksplit) v[s] = y[s * split_stride4 + (size_t)row * H4 + c];
        float4 a = v[0];
#pragma unroll
        for (int s = 1; s < kMaxSplit; ++s)
          if (s < ksplit) {
            a.x = __fadd_rn(a.x, v[s].x);
            a.y = __fadd_rn(a.y, v[s].y);
            a.z = __fadd_rn(a.z, v[s].z);
            a.w = __fadd_rn(a.w, v[s].w);
          }
        term[ty][cc][tx] = make_float4(__fmul_rn(g, a.x), __fmul_rn(g, a.y), __fmul_rn(g, a.z), __fmul_rn(g, a.w));
      }
    }
    __syncthreads();
    if (ty == 0) {
#pragma unroll
      for (int cc = 0; cc < kCombineChunks; ++cc)
        for (int i = 0; i < kCombineRows && j0 + i < J; ++i) {
          const float4 b = term[i][cc][tx];
          acc[cc].x = __fadd_rn(acc[cc].x, b.x);
          acc[cc].y = __fadd_rn(acc[cc].y, b.y);
          acc[cc].z = __fadd_rn(acc[cc].z, b.z);
          acc[cc].w = __fadd_rn(acc[cc].w, b.w);
        }
    }
    __syncthreads();
  }
  if (ty == 0) {
#pragma unroll
    for (int cc = 0; cc < kCombineChunks; ++cc) {
      const int c = c_first + cc * kCombineCols;
      if (c < H4) out[(size_t)t * H4 + c] = acc[cc];
    }
  }
}

// The same sum for batches with enough tokens to fill the machine by themselves: one thread per (token, float4
// column), U expert choices in flight at a time, no shared memory and no barrier.  The arithmetic and its order
// are those of combine_kernel (splits added in split order, times the gate, terms added in choice order).
template <int U>
__global__ void __launch_bounds__(128)
    combine_stream_kernel(const float4* y /* written by the kernel directly ahead */, const float* __restrict__ gates, const int32_t* __restrict__ inv_perm,
                          int T, int k, int n_shared, int H4, int ksplit, size_t split_stride4, float4* __restrict__ out) {
  grid_dep_sync();
  grid_dep_trigger();
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  const int t = blockIdx.y;
  if (c >= H4) return;
  const int J = k + n_shared;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int j0 = 0; j0 < J; j0 += U) {
    size_t row[U];
    float g[U];
    float4 a[U];
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const int j = j0 + i;
      if (j < k) {
        row[i] = (size_t)inv_perm[(size_t)t * k + j];
        g[i] = gates[(size_t)t * k + j];
      } else {
        row[i] = (size_t)T * k + (size_t)(j - k) * T + t;
        g[i] = 1.0f;
      }
    }
#pragma unroll
    for (int i = 0; i < U; ++i)
      if (j0 + i < J) a[i] = y[row[i] * H4 + c];
    for (int sp = 1; sp < ksplit; ++sp) {
      float4 v[U];
#pragma unroll
      for (int i = 0; i < U; ++i)
        if (j0 + i < J) v[i] = y[sp * split_stride4 + row[i] * H4 + c];
#pragma unroll
      for (int i = 0; i < U; ++i)
        if (j0 + i < J) {
          a[i].x = __fadd_rn(a[i].x, v[i].x);
          a[i].y = __fadd_rn(a[i].y, v[i].y);
          a[i].z = __fadd_rn(a[i].z, v[i].z);
          a[i].w = __fadd_rn(a[i].w, v[i].w);
        }
    }
#pragma unroll
    for (int i = 0; i < U; ++i)
      if (j0 + i < J) {
        acc.x = __fadd_rn(acc.x, __fmul_rn(g[i], a[i].x));
        acc.y = __fadd_rn(acc.y, __fmul_rn(g[i], a[i].y));
        acc.z = __fadd_rn(acc.z, __fmul_rn(g[i], a[i].z));
        acc.w = __fadd_rn(acc.w, __fmul_rn(g[i], a[i].w));
      }
  }
  out[(size_t)t * H4 + c] = acc;
}

pw_status launch_route(pw_ctx* ctx, int layer, const void* hidden, const float* logits, int T, int k, int nt_tile,
                       int ksplit, cudaStream_t s) {
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  char* b = ctx->base;
  const int E = c.n_experts, S = w.S;
  int32_t* ids = reinterpret_cast<int32_t*>(b + w.topk_ids);
  // a decode batch is routed by the grouping kernel's own CTA; a long prompt gets a grid of its own
  const bool fused = (long long)T * k * ((E + 31) / 32) <= kFusedRouteWork;
  timing_mark(ctx, PW_K_ROUTER, s);
  if (!fused) {
    PW_CUDA_OK(launch_dependent(router_kernel, dim3((T * 32 + 255) / 256), dim3(256), 0, s, logits, T, E, k, ids,
                                reinterpret_cast<float*>(b + w.gates)));
    ctx->launches += 1;
  }
  timing_mark(ctx, PW_K_PERMUTE, s);
  const size_t smem = sizeof(int32_t) * ((size_t)S + (S + 1) + E + 32 * (size_t)E + (S + 1) + S);
  const DevRow* rows = reinterpret_cast<const DevRow*>(b + w.table) + (size_t)layer * S * 3;
  PW_CUDA_OK(launch_dependent(
      permute_kernel, dim3(1), dim3(1024), smem, s, fused ? logits : static_cast<const float*>(nullptr),
      reinterpret_cast<float*>(b + w.gates), ids, T, k, E, c.n_shared, reinterpret_cast<int32_t*>(b + w.counts),
      reinterpret_cast<int32_t*>(b + w.offsets), reinterpret_cast<int32_t*>(b + w.perm),
      reinterpret_cast<int32_t*>(b + w.inv_perm), reinterpret_cast<int32_t*>(b + w.row_token),
      reinterpret_cast<int32_t*>(b + w.counter), rows, c.hidden, c.ffn, nt_tile, ksplit,
      reinterpret_cast<int2*>(b + w.tile_tab), w.max_tiles, reinterpret_cast<int32_t*>(b + w.n_units),
      reinterpret_cast<int32_t*>(b + w.seg_order), w.max_units, reinterpret_cast<int32_t*>(b + w.status)));
  const int R = T * k + c.n_shared * T;
  const int dn_tt_outer = (size_t)R * c.ffn * 2 > ((size_t)64 << 20) ? 1 : 0;   // SwiGLU rows beyond half of the L2
  timing_mark(ctx, PW_K_GATHER, s);
  dim3 grid((R + 255) / 256, (c.hidden / 8 + kGatherChunks - 1) / kGatherChunks);
  PW_CUDA_OK(launch_dependent(gather_kernel, grid, dim3(256), 0, s, reinterpret_cast<const uint4*>(hidden),
                              reinterpret_cast<const int32_t*>(b + w.row_token),
                              reinterpret_cast<const int32_t*>(b + w.offsets), S, c.hidden / 8, w.Rpad,
                              reinterpret_cast<uint4*>(b + w.xt), reinterpret_cast<const int32_t*>(b + w.counts),
                              reinterpret_cast<const int2*>(b + w.tile_tab), w.max_tiles,
                              reinterpret_cast<const int32_t*>(b + w.n_units), nt_tile, ksplit, c.hidden / kGroup,
                              c.ffn / kGroup, dn_tt_outer, reinterpret_cast<Unit*>(b + w.units_gu),
                              reinterpret_cast<Unit*>(b + w.units_dn), reinterpret_cast<int32_t*>(b + w.done)));
  ctx->launches += 2;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

pw_status launch_combine(pw_ctx* ctx, int T, int k, int ksplit, float* out, cudaStream_t s) {
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  char* b = ctx->base;
  const int H4 = c.hidden / 4;
  const int R = T * k + c.n_shared * T;
  const int chunks = T >= 256 ? 4 : 1;
  dim3 grid((H4 + kCombineCols * chunks - 1) / (kCombineCols * chunks), T);
  timing_mark(ctx, PW_K_COMBINE, s);
  if ((long long)T * ((H4 + 127) / 128) >= 2 * ctx->num_sms) {   // enough (token, column) CTAs to fill the machine
    PW_CUDA_OK(launch_dependent(combine_stream_kernel<4>, dim3((H4 + 127) / 128, T), dim3(128), 0, s,
                                reinterpret_cast<const float4*>(b + w.y), reinterpret_cast<const float*>(b + w.gates),
                                reinterpret_cast<const int32_t*>(b + w.inv_perm), T, k, c.n_shared, H4, ksplit,
                                (size_t)R * H4, reinterpret_cast<float4*>(out)));
    ctx->launches += 1;
    PW_CUDA_OK(cudaGetLastError());
    return PW_OK;
  }
  PW_CUDA_OK(launch_dependent(chunks == 4 ? combine_kernel<4> : combine_kernel<1>, grid, dim3(kCombineCols, kCombineRows), 0, s, reinterpret_cast<const float4*>(b + w.y),
                              reinterpret_cast<const float*>(b + w.gates),
                              reinterpret_cast<const int32_t*>(b + w.inv_perm), T, k, c.n_shared, H4, ksplit,
                              (size_t)R * H4, reinterpret_cast<float4*>(out)));
  ctx->launches += 1;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

}  // namespace pw

// ---- routing without any allocation ------------------------------------------------------------
// Scratch of pw_route_tokens_static: inverse permutation, operand-row map and counters of the
// grouping kernel.  Lives in the library image, so every GPU that loads the library holds it until
// the process exits.  In host code `g_route_scratch` is only a handle of the symbol, not a device
// address: the address a kernel may use comes from cudaGetSymbolAddress, once per device.
namespace {
constexpr int kStaticMaxPairs = 65536;        // T * top_k
constexpr int kStaticMaxExperts = 256;
constexpr size_t kStaticInvPerm = 0;                                            // int32[kStaticMaxPairs]
constexpr size_t kStaticRowToken = kStaticInvPerm + 4 * (size_t)kStaticMaxPairs;   // int32[kStaticMaxPairs + kPadRows]
constexpr size_t kStaticCounter = kStaticRowToken + 4 * (size_t)(kStaticMaxPairs + pw::kPadRows);   // int32[64]
constexpr size_t kStaticStatus = kStaticCounter + 256;                          // int32[64]
constexpr size_t kStaticBytes = kStaticStatus + 256;
static __device__ __align__(256) unsigned char g_route_scratch[kStaticBytes];
constexpr int kMaxDevices = 64;
static void* g_route_scratch_addr[kMaxDevices];   // device address of the array, per device, once resolved
}  // namespace

extern "C" pw_status pw_route_tokens_static(const float* router_logits, int T, int n_experts, int top_k,
                                            int32_t* topk_ids, float* gates, int32_t* counts, int32_t* offsets,
                                            int32_t* perm, pw_stream stream) {
  using namespace pw;
  if (!router_logits || !topk_ids || !gates || !counts || !offsets || !perm) return PW_ERR_INVALID_ARG;
  if (T < 1 || n_experts < 1 || top_k < 1 || top_k > n_experts || top_k > 32) return PW_ERR_INVALID_ARG;
  if (n_experts > kStaticMaxExperts || (long long)T * top_k > kStaticMaxPairs) return PW_ERR_NOMEM;
  const void* ptrs[6] = {router_logits, topk_ids, gates, counts, offsets, perm};
  for (const void* q : ptrs)
    if (reinterpret_cast<uintptr_t>(q) & 15) return PW_ERR_ALIGN;
  int dev = -1;
  PW_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return PW_ERR_INVALID_ARG;
  if (!g_route_scratch_addr[dev]) {   // first call on this device: resolve the symbol with this device current
    void* addr = nullptr;
    PW_CUDA_OK(cudaGetSymbolAddress(&addr, g_route_scratch));
    if (!addr) return PW_ERR_CUDA;
    g_route_scratch_addr[dev] = addr;
  }
  char* sc = reinterpret_cast<char*>(g_route_scratch_addr[dev]);
  router_kernel<<<(T * 32 + 255) / 256, 256, 0, stream>>>(router_logits, T, n_experts, top_k, topk_ids, gates);
  const int S = n_experts;
  const size_t smem = sizeof(int32_t) * ((size_t)S + (S + 1) + n_experts + 32 * (size_t)n_experts + (S + 1) + S);
  // the grouping kernel clears the counters it uses; everything else in the scratch is overwritten before it is read
  permute_kernel<<<1, 1024, smem, stream>>>(nullptr, nullptr, topk_ids, T, top_k, n_experts, 0, counts, offsets, perm,
                                            reinterpret_cast<int32_t*>(sc + kStaticInvPerm),
                                            reinterpret_cast<int32_t*>(sc + kStaticRowToken),
                                            reinterpret_cast<int32_t*>(sc + kStaticCounter), nullptr, 0, 0, 0, 1, nullptr,
                                            0, nullptr, nullptr, 0,
                                            reinterpret_cast<int32_t*>(sc + kStaticStatus));
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

