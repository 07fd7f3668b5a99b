// Tensor-core expert FFN for sm_100a: weight pages stream HBM -> shared memory (bulk async copies),
// are dequantized in registers straight into tensor memory (the A operand, one weight row per TMEM
// lane), and tcgen05.mma contracts them against the token tile (B operand in shared memory), with
// fp32 accumulators in tensor memory.  D[128 weight rows, N tokens] += W[128, 16] * X[N, 16]^T.
//
// One persistent CTA per SM, 10 warps:
//   warps 0-7  dequantize (two sets of four warps alternate groups; warp w owns TMEM lanes
//              32*(w%4) .. +31) and run the epilogue (SwiGLU -> fp16 operand of the down projection,
//              or the fp32 partial output of the down projection);
//   warp 8     producer: one thread issues every bulk copy (weight stages and token tiles);
//   warp 9     allocates tensor memory; one thread issues every MMA and commit.
// Every wait on an mbarrier is bounded; when one runs out the CTA records PW_ERR_TIMEOUT in the
// status word, stops issuing work, frees its tensor memory and returns.
#include "pw_common.cuh"
#include "pw_layout.cuh"

namespace pw {

constexpr int kWSlots = 4;                     // weight stages in shared memory
constexpr int kWSlotCodes = 32768;             // code bytes of a stage (16 units x 2 KB)
constexpr int kWSlotMeta = 2048;               // scale bytes, then zero-point bytes, of up to 8 groups
constexpr int kWSlotBytes = kWSlotCodes + 2 * kWSlotMeta;
constexpr int kASlots = 4;                     // dequantized groups in tensor memory (64 columns each)
constexpr int kMaxBSlots = 4;
constexpr int kCtrlBytes = 1024;
constexpr int kMaxDynSmem = 232448;            // 227 KB
constexpr int kThreads = 320;
constexpr int kTmemCols = 512;
constexpr uint32_t kColD0 = 0, kColD1 = 128, kColA = 256;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // 2 s

struct Ctrl {                                  // lives at the start of dynamic shared memory
  unsigned long long w_full[kWSlots], w_empty[kWSlots];
  unsigned long long b_full[kMaxBSlots], b_empty[kMaxBSlots];
  unsigned long long a_full[kASlots], a_empty[kASlots];
  unsigned long long d_full, d_empty;
  uint32_t tmem_base;
  volatile int abort_flag;
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(unsigned long long* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(unsigned long long* b, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(b)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long globaltimer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false when the CTA is aborting or the limit ran out (and then raises the abort).
__device__ __forceinline__ bool mbar_wait(unsigned long long* b, uint32_t parity, Ctrl* c, int32_t* status) {
  if (mbar_try(b, parity)) return true;
  const unsigned long long t0 = globaltimer();
  uint32_t spins = 0;
  while (true) {
    if (mbar_try(b, parity)) return true;
    if (c->abort_flag) return false;
    if ((++spins & 1023u) == 0 && globaltimer() - t0 > kWaitLimitNs) {
      c->abort_flag = 1;
      atomicMax(status, (int)PW_ERR_TIMEOUT);
      return false;
    }
  }
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(unsigned long long* b) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(b))
               : "memory");
}
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const __half2* v) {
  const uint32_t* r = reinterpret_cast<const uint32_t*>(v);
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]), "r"(r[16]), "r"(r[17]), "r"(r[18]),
      "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]), "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]),
      "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// groups per weight stage: about 32 KB of codes whatever the bitwidth
__device__ __forceinline__ int groups_per_stage(uint32_t bits) { return bits == 16 ? 1 : bits == 8 ? 2 : bits == 2 ? 8 : 4; }

// Shared-memory matrix descriptor of the B operand: K-major, no swizzle.  A core matrix is 8 token
// rows x 16 bytes (8 fp16 along K) stored as 128 contiguous bytes; 8-row groups are 128 bytes apart
// (stride byte offset), the two K-halves of one MMA are `lbo_bytes` apart (leading byte offset).
__device__ __forceinline__ uint64_t make_b_desc(uint32_t saddr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((128u >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of sm_100
  return d;
}

template <int BITS>
__device__ __forceinline__ void dequant_group_to_tmem(const char* slot, int sub, int r, uint32_t taddr) {
  const uint4* row_units = reinterpret_cast<const uint4*>(slot + (size_t)sub * tile_code_bytes(BITS)) + r;
  __half2 s2 = u32_as_h2(0x3c003c00u), z2 = s2;
  if constexpr (BITS < 16) {
    s2 = __half2half2(reinterpret_cast<const __half*>(slot + kWSlotCodes)[sub * kTileRows + r]);
    z2 = __half2half2(reinterpret_cast<const __half*>(slot + kWSlotCodes + kWSlotMeta)[sub * kTileRows + r]);
  }
  __half2 w[32];
  decode_half<BITS>(row_units, 0, s2, z2, w);
  tmem_st32(taddr, w);
  decode_half<BITS>(row_units, 1, s2, z2, w);
  tmem_st32(taddr + 32, w);
}

// PHASE 0: units of (expert, 128 FFN rows, token tile): gate and up pages -> Ht.
// PHASE 1: units of (expert, 128 hidden rows, token tile, K range): down page -> Y[split].
template <int PHASE>
__global__ void __launch_bounds__(kThreads, 1) ffn_tc_kernel(const DevRow* __restrict__ rows, const Unit* __restrict__ units,
                                                             const int32_t* __restrict__ n_units_ptr,
                                                             const uint4* __restrict__ bop, int Rpad, int nt_tile,
                                                             int n_bslots, __half* __restrict__ ht,
                                                             float* __restrict__ y, int H, size_t y_split_stride,
                                                             int32_t* __restrict__ status) {
  extern __shared__ __align__(1024) char smem[];
  Ctrl* c = reinterpret_cast<Ctrl*>(smem);
  char* wslots = smem + kCtrlBytes;
  char* bslots = wslots + kWSlots * kWSlotBytes;
  const int bslot_bytes = nt_tile * 256;
  constexpr int NMAT = PHASE == 0 ? 2 : 1;
  constexpr int RING = kWSlots / NMAT;           // stages per matrix ring
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_units = n_units_ptr[PHASE];

  if (threadIdx.x == 0) {
    for (int i = 0; i < kWSlots; ++i) {
      mbar_init(&c->w_full[i], 1);
      mbar_init(&c->w_empty[i], 8);
    }
    for (int i = 0; i < kMaxBSlots; ++i) {
      mbar_init(&c->b_full[i], 1);
      mbar_init(&c->b_empty[i], 1);
    }
    for (int i = 0; i < kASlots; ++i) {
      mbar_init(&c->a_full[i], 4);
      mbar_init(&c->a_empty[i], 1);
    }
    mbar_init(&c->d_full, 1);
    mbar_init(&c->d_empty, 8);
    c->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = c->tmem_base;

  if (warp == 8) {
    // ---------------- producer ----------------
    if (lane == 0) {
      uint32_t wcount[NMAT] = {};   // stages issued per ring
      uint32_t bcount = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
        const Unit un = units[u];
        const DevRow* rr = rows + un.seg * 3;
        const int nb_rows = (un.ntok + 15) & ~15;
        for (int g = un.g0; ok && g < un.g1; ++g) {
          {  // token tile of this group: 16 K-chunks of nb_rows x 16 bytes
            const int bs = bcount % n_bslots;
            ok = mbar_wait(&c->b_empty[bs], ((bcount / n_bslots) & 1) ^ 1, c, status);
            if (!ok) break;
            mbar_expect_tx(&c->b_full[bs], nb_rows * 256);
            char* dst = bslots + (size_t)bs * bslot_bytes;
            const uint4* src = bop + (size_t)(g * 16) * Rpad + un.tok0;
            for (int kc = 0; kc < 16; ++kc)
              bulk_g2s(dst + kc * nb_rows * 16, src + (size_t)kc * Rpad, nb_rows * 16, &c->b_full[bs]);
            ++bcount;
          }
#pragma unroll
          for (int m = 0; m < NMAT; ++m) {
            const DevRow& row = rr[PHASE == 0 ? m : 2];
            const int gps = groups_per_stage(row.bits);
            if ((g - un.g0) % gps != 0) continue;
            const int ngr = min(gps, un.g1 - g);
            const int ws = m * RING + (int)(wcount[m] % RING);
            ok = mbar_wait(&c->w_empty[ws], ((wcount[m] / RING) & 1) ^ 1, c, status);
            if (!ok) break;
            const int ng = row.cols / kGroup;
            const size_t tile = (size_t)un.row_tile * ng + g;
            const uint32_t cbytes = ngr * row.bits * 2048;
            const uint32_t mbytes = row.bits < 16 ? ngr * 256 : 0;
            mbar_expect_tx(&c->w_full[ws], cbytes + 2 * mbytes);
            char* dst = wslots + (size_t)ws * kWSlotBytes;
            bulk_g2s(dst, reinterpret_cast<const char*>(row.codes) + tile * row.bits * 2048, cbytes, &c->w_full[ws]);
            if (mbytes) {
              bulk_g2s(dst + kWSlotCodes, row.scales + tile * kTileRows, mbytes, &c->w_full[ws]);
              bulk_g2s(dst + kWSlotCodes + kWSlotMeta, row.zps + tile * kTileRows, mbytes, &c->w_full[ws]);
            }
            ++wcount[m];
          }
        }
      }
      if (!ok) {
        // let copies already in flight land before the CTA leaves (bounded)
        const unsigned long long t0 = globaltimer();
        while (globaltimer() - t0 < 200000ull) {
        }
      }
    }
  } else if (warp == 9) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      uint32_t acount = 0, bcount = 0, ucount = 0;
      bool ok = true;
      for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x, ++ucount) {
        const Unit un = units[u];
        const int nb_rows = (un.ntok + 15) & ~15;
        const uint32_t idesc = (1u << 4) | ((uint32_t)(nb_rows >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        ok = mbar_wait(&c->d_empty, (ucount & 1) ^ 1, c, status);   // epilogue of the previous unit is done
        if (!ok) break;
        tc_fence_after();
        for (int g = un.g0; ok && g < un.g1; ++g) {
          const int bs = bcount % n_bslots;
          ok = mbar_wait(&c->b_full[bs], (bcount / n_bslots) & 1, c, status);
          if (!ok) break;
          const uint32_t baddr = smem_u32(bslots + (size_t)bs * bslot_bytes);
#pragma unroll
          for (int m = 0; m < NMAT; ++m) {
            const int as = acount % kASlots;
            ok = mbar_wait(&c->a_full[as], (acount / kASlots) & 1, c, status);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_t = tmem + (m == 0 ? kColD0 : kColD1);
            const uint32_t a_t = tmem + kColA + as * 64;
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {
              const uint64_t bd = make_b_desc(baddr + kk * 2 * nb_rows * 16, nb_rows * 16);
              tc_mma_ts(d_t, a_t + kk * 8, bd, idesc, (g > un.g0 || kk > 0) ? 1u : 0u);
            }
            tc_commit(&c->a_empty[as]);
            ++acount;
          }
          if (!ok) break;
          tc_commit(&c->b_empty[bs]);
          ++bcount;
        }
        if (ok) tc_commit(&c->d_full);
      }
    }
  } else {
    // ---------------- dequantize + epilogue (warps 0..7) ----------------
    const int set = warp >> 2, q = warp & 3;
    const int r = q * 32 + lane;                     // weight row inside the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t wcount[NMAT] = {};
    uint32_t acount = 0, ucount = 0;
    bool ok = true;
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x, ++ucount) {
      const Unit un = units[u];
      const DevRow* rr = rows + un.seg * 3;
      for (int g = un.g0; ok && g < un.g1; ++g) {
#pragma unroll
        for (int m = 0; m < NMAT; ++m) {
          const uint32_t bits = rr[PHASE == 0 ? m : 2].bits;
          const int gps = groups_per_stage(bits);
          const int sub = (g - un.g0) % gps;
          const int ws = m * RING + (int)(wcount[m] % RING);
          if (sub == 0) {
            ok = mbar_wait(&c->w_full[ws], (wcount[m] / RING) & 1, c, status);
            if (!ok) break;
          }
          const int as = acount % kASlots;
          if ((int)(acount & 1) == set) {
            ok = mbar_wait(&c->a_empty[as], ((acount / kASlots) & 1) ^ 1, c, status);
            if (!ok) break;
            tc_fence_after();
            const char* slot = wslots + (size_t)ws * kWSlotBytes;
            const uint32_t taddr = lane_addr + kColA + as * 64;
            switch (bits) {
              case 16: dequant_group_to_tmem<16>(slot, sub, r, taddr); break;
              case 8: dequant_group_to_tmem<8>(slot, sub, r, taddr); break;
              case 4: dequant_group_to_tmem<4>(slot, sub, r, taddr); break;
              case 3: dequant_group_to_tmem<3>(slot, sub, r, taddr); break;
              default: dequant_group_to_tmem<2>(slot, sub, r, taddr); break;
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&c->a_full[as]);
          }
          ++acount;
          if (sub == gps - 1 || g == un.g1 - 1) {     // last group of this stage: hand the slot back
            __syncwarp();
            if (lane == 0) mbar_arrive(&c->w_empty[ws]);
            ++wcount[m];
          }
        }
      }
      if (!ok) break;
      // ---- epilogue of the unit ----
      ok = mbar_wait(&c->d_full, ucount & 1, c, status);
      if (!ok) break;
      tc_fence_after();
      const int nb_rows = (un.ntok + 15) & ~15;
      const int half_cols = nb_rows >> 1;              // multiple of 8
      const int row = un.row_tile * kTileRows + r;
      for (int c0 = set * half_cols; c0 < (set + 1) * half_cols; c0 += 8) {
        float a[8], b[8];
        tmem_ld8(lane_addr + kColD0 + c0, a);
        if (PHASE == 0) tmem_ld8(lane_addr + kColD1 + c0, b);
        tmem_wait_ld();
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int n = c0 + i;
          if (n < un.ntok) {
            if (PHASE == 0) {
              const float hval = __fmul_rn(__fdiv_rn(a[i], __fadd_rn(1.0f, expf(-a[i]))), b[i]);
              ht[((size_t)(row >> 3) * Rpad + un.tok0 + n) * 8 + (row & 7)] = __float2half_rn(hval);
            } else {
              y[(size_t)un.split * y_split_stride + (size_t)(un.tok0 + n) * H + row] = a[i];
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&c->d_empty);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

int tensor_token_tile(const pw_ctx* ctx, int T, int k) {
  (void)ctx;
  (void)k;
  // an expert never holds more than T tokens; tiles of at most 128 tokens (two fp32 accumulators of
  // 128 columns plus four 64-column operand slots fill the 512 tensor-memory columns)
  int nt = (T + 15) & ~15;
  if (nt > 128) nt = 128;
  return nt;
}

pw_status launch_ffn_tensor(pw_ctx* ctx, int layer, int T, int k, int nt_tile, int ksplit, cudaStream_t s) {
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  char* b = ctx->base;
  const DevRow* rows = reinterpret_cast<const DevRow*>(b + w.table) + (size_t)layer * w.S * 3;
  const int bslot_bytes = nt_tile * 256;
  int n_bslots = (kMaxDynSmem - kCtrlBytes - kWSlots * kWSlotBytes) / bslot_bytes;
  if (n_bslots > kMaxBSlots) n_bslots = kMaxBSlots;
  if (n_bslots < 2) return PW_ERR_NOMEM;
  const int smem = kCtrlBytes + kWSlots * kWSlotBytes + n_bslots * bslot_bytes;
  if (!ctx->tc_state) {
    PW_CUDA_OK(cudaFuncSetAttribute(ffn_tc_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    PW_CUDA_OK(cudaFuncSetAttribute(ffn_tc_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    ctx->tc_state = ctx;
  }
  const int R = T * k + c.n_shared * T;
  int32_t* status = reinterpret_cast<int32_t*>(b + w.status);
  const int32_t* n_units = reinterpret_cast<const int32_t*>(b + w.n_units);
  timing_mark(ctx, PW_K_FFN_GATE_UP, s);
  ffn_tc_kernel<0><<<ctx->num_sms, kThreads, smem, s>>>(rows, reinterpret_cast<const Unit*>(b + w.units_gu), n_units,
                                                        reinterpret_cast<const uint4*>(b + w.xt), w.Rpad, nt_tile,
                                                        n_bslots, reinterpret_cast<__half*>(b + w.ht), nullptr,
                                                        c.hidden, 0, status);
  timing_mark(ctx, PW_K_FFN_DOWN, s);
  ffn_tc_kernel<1><<<ctx->num_sms, kThreads, smem, s>>>(rows, reinterpret_cast<const Unit*>(b + w.units_dn), n_units,
                                                        reinterpret_cast<const uint4*>(b + w.ht), w.Rpad, nt_tile,
                                                        n_bslots, nullptr, reinterpret_cast<float*>(b + w.y), c.hidden,
                                                        (size_t)R * c.hidden, status);
  ctx->launches += 2;
  PW_CUDA_OK(cudaGetLastError());
  (void)ksplit;
  return PW_OK;
}

}  // namespace pw
