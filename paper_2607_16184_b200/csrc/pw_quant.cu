// Group-wise quantize / demote of a linear-block into a weight page, and the TILED <-> CANONICAL
// layout conversions.  One CTA per (128-row, one-group) tile, four threads per row, each owning a
// 32-weight slice; HBM-bound: reads the source once, writes the page once.
#include "pw_common.cuh"
#include "pw_layout.cuh"
#include "pw_quant_core.cuh"

namespace pw {

enum SrcKind { SRC_RAW = 0, SRC_TILED = 1 };

// The fp16 weight a stored code stands for, bit for bit: fp32 product (exact), fp32 add, one
// rounding to fp16.
__device__ __forceinline__ float dequant_exact(int code, float s, float z) {
  return __half2float(__float2half_rn(__fadd_rn(__fmul_rn((float)code, s), z)));
}


// Words of slice q of row r of a tile image, fetched with the widest loads the layout allows.
template <int BITS>
__device__ __forceinline__ void load_slice_words(const char* tb, int r, int q, uint32_t* w) {
  if constexpr (BITS == 16 || BITS == 8 || BITS == 4) {
    constexpr int NU = BITS == 16 ? 4 : BITS == 8 ? 2 : 1;
#pragma unroll
    for (int i = 0; i < NU; ++i) {
      const uint4 u = __ldg(reinterpret_cast<const uint4*>(tb + slice_word_offset<BITS>(r, q, 4 * i)));
      w[4 * i] = u.x;
      w[4 * i + 1] = u.y;
      w[4 * i + 2] = u.z;
      w[4 * i + 3] = u.w;
    }
  } else {
    const uint2 u = __ldg(reinterpret_cast<const uint2*>(tb + slice_word_offset<BITS>(r, q, 0)));
    w[0] = u.x;
    w[1] = u.y;
    if constexpr (BITS == 3) w[2] = __ldg(reinterpret_cast<const uint32_t*>(tb + slice_word_offset<3>(r, q, 2)));
  }
}

// Words of my slice of tile (rt, g) of the source, as they lie in memory (an fp16 matrix or a tile image).
template <int SRC_KIND, int SRC_BITS>
__device__ __forceinline__ void load_source_slice(const void* __restrict__ src_codes, uint32_t cols, int rt, int g, int ng,
                                                  int r, int q, uint32_t* raw) {
  if constexpr (SRC_KIND == SRC_RAW) {
    const uint4* p = reinterpret_cast<const uint4*>(reinterpret_cast<const __half*>(src_codes) +
                                                    ((size_t)rt * kTileRows + r) * cols + (size_t)g * kGroup + 32 * q);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint4 u = __ldg(p + i);
      raw[4 * i] = u.x;
      raw[4 * i + 1] = u.y;
      raw[4 * i + 2] = u.z;
      raw[4 * i + 3] = u.w;
    }
  } else {
    const char* tb = reinterpret_cast<const char*>(src_codes) + ((size_t)rt * ng + g) * tile_bytes(SRC_BITS);
    load_slice_words<SRC_BITS>(tb, r, q, raw);
  }
}

// NT: tiles per CTA (group g and, NT == 2, group g + n_groups / 2 of the same row tile).  The loads of all of
// them are issued before the first is worked on: twice the bytes in flight per thread, and the second tile's
// latency is covered by the first one's arithmetic.
template <int SRC_KIND, int SRC_BITS, int DST_BITS, int NT>
__global__ void __launch_bounds__(512, NT == 2 ? 2 : 3) quant_tile_kernel(const void* __restrict__ src_codes, uint32_t cols,
                                                                          void* __restrict__ dst_codes) {
  const int rt = blockIdx.y, ng = gridDim.x * NT;
  const int r = threadIdx.x >> 2, q = threadIdx.x & 3;
  constexpr int NWS = SliceWords<SRC_BITS>::kWords;
  uint32_t raw[NT][NWS];
#pragma unroll
  for (int k = 0; k < NT; ++k)
    load_source_slice<SRC_KIND, SRC_BITS>(src_codes, cols, rt, blockIdx.x + k * gridDim.x, ng, r, q, raw[k]);

#pragma unroll
  for (int k = 0; k < NT; ++k) {
  const int g = blockIdx.x + k * gridDim.x;
  const size_t tile = (size_t)rt * ng + g;
  float v[32];
  __half2 h16[SRC_BITS == 16 ? 16 : 1];             // the packed halves of a 16-bit source
  if constexpr (SRC_BITS == 16) {
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      h16[i] = u32_as_h2(raw[k][i]);
      const float2 f = __half22float2(h16[i]);
      v[2 * i] = f.x;
      v[2 * i + 1] = f.y;
    }
  } else {
    const char* tb = reinterpret_cast<const char*>(src_codes) + tile * tile_bytes(SRC_BITS);
    int code[32];
    unpack_slice<SRC_BITS>(raw[k], code);
    const float s = __half2float(*reinterpret_cast<const __half*>(tb + tile_scale_offset(SRC_BITS, r)));
    const float z = __half2float(*reinterpret_cast<const __half*>(tb + tile_zp_offset(SRC_BITS, r)));
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = dequant_exact(code[i], s, z);
  }

  char* db = reinterpret_cast<char*>(dst_codes) + tile * tile_bytes(DST_BITS);
  if constexpr (DST_BITS == 16) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint4 o;
      __half2* h = reinterpret_cast<__half2*>(&o);
#pragma unroll
      for (int j = 0; j < 4; ++j) h[j] = __floats2half2_rn(v[8 * i + 2 * j], v[8 * i + 2 * j + 1]);
      *reinterpret_cast<uint4*>(db + slice_word_offset<16>(r, q, 4 * i)) = o;
    }
  } else {
  int code[32];
  __half sh;
  float lo;
  constexpr int NW = SliceWords<DST_BITS>::kWords;
  uint32_t w[NW];
  if constexpr (DST_BITS == 3) {
    group_quantize<SRC_BITS == 16>(v, h16, (1 << DST_BITS) - 1, code, sh, lo);
    pack_slice<DST_BITS>(code, w);
  } else {                                           // the upper clamp of the codes is the pack's saturation
    group_quantize<SRC_BITS == 16, false>(v, h16, (1 << DST_BITS) - 1, code, sh, lo);
    pack_slice_sat<DST_BITS>(code, w);
  }
  if constexpr (DST_BITS == 8) {
    *reinterpret_cast<uint4*>(db + slice_word_offset<8>(r, q, 0)) = make_uint4(w[0], w[1], w[2], w[3]);
    *reinterpret_cast<uint4*>(db + slice_word_offset<8>(r, q, 4)) = make_uint4(w[4], w[5], w[6], w[7]);
  } else if constexpr (DST_BITS == 4) {
    *reinterpret_cast<uint4*>(db + slice_word_offset<4>(r, q, 0)) = make_uint4(w[0], w[1], w[2], w[3]);
  } else {
    *reinterpret_cast<uint2*>(db + slice_word_offset<DST_BITS>(r, q, 0)) = make_uint2(w[0], w[1]);
    if constexpr (DST_BITS == 3) *reinterpret_cast<uint32_t*>(db + slice_word_offset<3>(r, q, 2)) = w[2];
  }
  if (q == 0) {
    *reinterpret_cast<__half*>(db + tile_scale_offset(DST_BITS, r)) = sh;
    *reinterpret_cast<__half*>(db + tile_zp_offset(DST_BITS, r)) = __float2half_rn(lo);
  }
  }
  }
}

// 4 bits -> 3 or 2 bits without touching a weight.  A group has at most 16 distinct values, one per source code,
// and the demote Q(D(.)) is a function of the code alone: minimum and maximum are the values of the smallest and
// the largest code present, and new_code(c) = clamp(rint((D(c) - lo) / scale')) is non-decreasing in c.  One thread
// owns a whole group (a row of a tile: 16 words), so the group's work is done once and not by each of four lanes:
// it evaluates the general kernel's arithmetic, bit for bit, on the 16 codes, turns the table into L thresholds
// t_k = number of source codes whose new code is below k, and every code becomes [c >= t_1] + .. + [c >= t_L]:
// one add and one three-input logic operation per threshold compare all eight nibbles of a code word at once, and
// because the comparisons are nested a few more logic operations give the bits of their count.
constexpr int kRequantThreads = 256;              // two tiles per CTA
template <int DB>
__global__ void __launch_bounds__(kRequantThreads) requant_from4_kernel(const void* __restrict__ src_codes, uint32_t n_tiles,
                                                                        void* __restrict__ dst_codes) {
  const int r = threadIdx.x & (kTileRows - 1);
  const size_t tile = (size_t)blockIdx.x * (kRequantThreads / kTileRows) + (threadIdx.x >> 7);
  if (tile >= n_tiles) return;
  const char* tb = reinterpret_cast<const char*>(src_codes) + tile * tile_bytes(4);
  uint32_t w[16];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(tb + slice_word_offset<4>(r, q, 0)));
    w[4 * q] = u.x;
    w[4 * q + 1] = u.y;
    w[4 * q + 2] = u.z;
    w[4 * q + 3] = u.w;
  }
  const float s = __half2float(*reinterpret_cast<const __half*>(tb + tile_scale_offset(4, r)));
  const float z = __half2float(*reinterpret_cast<const __half*>(tb + tile_zp_offset(4, r)));

  // smallest and largest code of the group: a page written by the quantizer always uses 0 and 15 (the extremes
  // of the group map to them), which two zero-nibble tests see (bit 3 of a nibble of x - 0x1111.. & ~x is set for
  // the lowest zero nibble of x; ~x - k = ~(x + k)); any other page takes the exact scan
  uint32_t has0 = 0, has15 = 0;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    has0 |= (w[i] - 0x11111111u) & ~w[i];
    has15 |= ~(w[i] + 0x11111111u) & w[i];
  }
  int cmin = 0, cmax = 15;
  if (((has0 & 0x88888888u) == 0) | ((has15 & 0x88888888u) == 0)) {
    int mn = 15, mx = 0;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int c = (int)((w[i] >> (4 * j)) & 15u);
        mn = min(mn, c);
        mx = max(mx, c);
      }
    }
    cmin = mn;
    cmax = mx;
  }

  // scale and zero-point of the new page: the general quantizer's arithmetic on the two extreme values
  constexpr int L = (1 << DB) - 1;
  float lo = dequant_exact(cmin, s, z);
  const float hi = dequant_exact(cmax, s, z);
  if (lo == 0.0f) lo = 0.0f;  // store -0 as +0
  const float rng = __fsub_rn(hi, lo);
  __half sh;
  if (rng == 0.0f) {
    sh = __ushort_as_half((unsigned short)0x3c00);
  } else {
    sh = __float2half_rn(__fdiv_rn(rng, (float)L));
    if ((__half_as_ushort(sh) & 0x7fff) == 0) sh = __ushort_as_half((unsigned short)0x0001);
  }
  const float rinv = __fdiv_rn(1.0f, __half2float(sh));

  // t_k = how many of the 16 source codes get a new code below k = 16 - (codes that reach k).  The new code is
  // min(rint(x), L) with x = (D(c) - lo) * rinv (negative for a code below the smallest one present: new code 0;
  // NaN when the source's largest value overflowed fp16: new code 0 as well, as the conversion to an integer of
  // the general kernel gives), and with ties to even rint(x) >= k  <=>  x > k - 0.5 (k odd), x >= k - 0.5 (k even),
  // the latter being x > the float just below k - 0.5.  Each comparison x > e is one saturating multiply-add --
  // sat((x - e) * 2^40) is 1 for x > e and 0 otherwise (also for NaN); the rounding of the sum keeps sign and
  // zero-ness -- and one add, both on the multiply-add pipe that the logic operations below leave idle.
  float reach[L];
#pragma unroll
  for (int k = 0; k < L; ++k) reach[k] = 0.0f;
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    const float x = __fmul_rn(__fsub_rn(dequant_exact(c, s, z), lo), rinv);
#pragma unroll
    for (int k = 1; k <= L; ++k) {
      constexpr float kBig = 1099511627776.0f;     // 2^40
      const float edge = (float)k - 0.5f;
      const float ulp = edge >= 4.0f ? 4.76837158203125e-7f : edge >= 2.0f ? 2.384185791015625e-7f : 1.1920928955078125e-7f;
      const float e = (k & 1) ? edge : edge - ulp;
      reach[k - 1] += __saturatef(fmaf(x, kBig, -e * kBig));
    }
  }
  // The comparison c >= t_k on all eight nibbles of a word at once.  With c = 8 h + l: for t <= 8 it is
  // h | (l >= t), for t > 8 it is h & (l >= t - 8), and l >= t' (0 <= t' <= 8) is bit 3 of l + (8 - t'), which never
  // carries out of the nibble.  So per threshold one add on the word with the h bits masked out, and one majority
  // function of (sum, word, m_k) -- m_k all ones for t_k <= 8 (or), zero above (and) -- leave the flag in bit 3 of
  // every nibble.  With n = 16 - t codes reaching k: 8 - t' = n - 8 for n >= 8, n below.
  uint32_t kk[L], mk[L];
#pragma unroll
  for (int k = 0; k < L; ++k) {
    const uint32_t n = __float2uint_rn(reach[k]);
    kk[k] = (n >= 8u ? n - 8u : n) * 0x11111111u;
    mk[k] = n >= 8u ? 0xffffffffu : 0u;
  }

  uint32_t half_bytes[16];                         // per source word: the 2-bit codes of 8 weights, a byte in each half-word
  uint32_t third[4];                               // DB == 3, per slice: the plane of the third bits (plane_bit_pos)
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if ((i & 3) == 0) third[i >> 2] = 0;
    const uint32_t low = w[i] & 0x77777777u;
    uint32_t f[L];
#pragma unroll
    for (int k = 0; k < L; ++k) asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(f[k]) : "r"(low + kk[k]), "r"(w[i]), "r"(mk[k]));
    // the comparisons are nested (t_1 <= t_2 <= ..), so bit 0 of their count is ((f1 & ~f2) | f3) & ~f4 | .. and
    // bit 1 is (f2 & ~f4) | f6, bit 2 is f4 -- all in bit 3 of every nibble
    uint32_t b0, b1;
    asm("lop3.b32 %0, %1, %2, %3, 0xBA;" : "=r"(b0) : "r"(f[0]), "r"(f[1]), "r"(f[2]));
    if constexpr (DB == 3) {
      asm("lop3.b32 %0, %1, %2, %3, 0xBA;" : "=r"(b0) : "r"(b0), "r"(f[3]), "r"(f[4]));
      asm("lop3.b32 %0, %1, %2, %3, 0xBA;" : "=r"(b0) : "r"(b0), "r"(f[5]), "r"(f[6]));
      asm("lop3.b32 %0, %1, %2, %3, 0xBA;" : "=r"(b1) : "r"(f[1]), "r"(f[3]), "r"(f[5]));
      // third bits: nibble a of the word (flag in bit 4 a + 3) -> bit a of its half-word.  Moved to bit 4 a + 1, the
      // shifts by 1, 4, 7, 10 bring a = 0 .. 3 to bits 0 .. 3 and no two copies share a bit (4 a - 3 j is different
      // for every a and j): one high product.  The plane keeps the four pairs of source word i at every other
      // bit from plane_bit_pos(4 (i mod 4)) on, so the four bits are spread to every other place first.
      const uint32_t g = __umulhi((f[3] >> 2) & 0x22222222u, (1u << 31) + (1u << 28) + (1u << 25) + (1u << 22));
      uint32_t sp = g & 0x000f000fu;
      sp = (sp | (sp << 2)) & 0x00330033u;
      sp = (sp | (sp << 1)) & 0x00550055u;
      third[i >> 2] |= sp << plane_bit_pos(4 * (i & 3));
    } else {
      b1 = f[1];
    }
    // low two bits of every new code into the low bits of its nibble, then the four codes of a half-word into its
    // low byte (what lands in the upper byte is dropped by the byte permute below)
    const uint32_t t = and_or(b0 >> 3, 0x11111111u, (b1 >> 2) & 0x22222222u);
    const uint32_t u = (t | (t >> 2)) & 0x0f0f0f0fu;
    half_bytes[i] = u | (u >> 4);
  }
  // slices 2h and 2h + 1 of a row share a 16-byte chunk of the destination tile
  char* db = reinterpret_cast<char*>(dst_codes) + tile * tile_bytes(DB);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const uint32_t* hb = half_bytes + 8 * h;
    *reinterpret_cast<uint4*>(db + slice_word_offset<DB>(r, 2 * h, 0)) =
        make_uint4(__byte_perm(hb[0], hb[1], 0x6240), __byte_perm(hb[2], hb[3], 0x6240), __byte_perm(hb[4], hb[5], 0x6240),
                   __byte_perm(hb[6], hb[7], 0x6240));
  }
  if constexpr (DB == 3)
    *reinterpret_cast<uint4*>(db + slice_word_offset<3>(r, 0, 2)) = make_uint4(third[0], third[1], third[2], third[3]);
  *reinterpret_cast<__half*>(db + tile_scale_offset(DB, r)) = sh;
  *reinterpret_cast<__half*>(db + tile_zp_offset(DB, r)) = __float2half_rn(lo);
}

// TILED -> CANONICAL (EXPORT = true) or CANONICAL -> TILED, same bitwidth.
template <int BITS, bool EXPORT>
__global__ void __launch_bounds__(512) relayout_kernel(const void* __restrict__ src_codes, uint32_t cols,
                                                       void* __restrict__ dst_codes,
                                                       __half* __restrict__ can_scales,   // canonical side
                                                       __half* __restrict__ can_zps) {
  const int g = blockIdx.x, rt = blockIdx.y, ng = gridDim.x;
  const int r = threadIdx.x >> 2, q = threadIdx.x & 3;
  const size_t tile = (size_t)rt * ng + g;
  const size_t row = (size_t)rt * kTileRows + r;
  const size_t elem = row * cols + (size_t)g * kGroup + 32 * q;   // first element of the slice
  constexpr int NW = SliceWords<BITS>::kWords;
  // canonical side: the slice is BITS words of the bit stream (fp16: 16 words of the matrix)
  const char* csrc = reinterpret_cast<const char*>(EXPORT ? dst_codes : src_codes);
  char* cpos = const_cast<char*>(csrc) + elem * BITS / 8;
  const char* tsrc = reinterpret_cast<const char*>(EXPORT ? src_codes : dst_codes);
  char* tpos = const_cast<char*>(tsrc) + tile * tile_bytes(BITS);

  uint32_t w[NW];
  if constexpr (EXPORT) {
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = *reinterpret_cast<const uint32_t*>(tpos + slice_word_offset<BITS>(r, q, i));
    if constexpr (BITS == 16) {
#pragma unroll
      for (int i = 0; i < 16; ++i) reinterpret_cast<uint32_t*>(cpos)[i] = w[i];
    } else {
      int code[32];
      unpack_slice<BITS>(w, code);
      unsigned long long acc = 0;
      int nb = 0, wi = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        acc |= (unsigned long long)code[i] << nb;
        nb += BITS;
        if (nb >= 32) {
          reinterpret_cast<uint32_t*>(cpos)[wi++] = (uint32_t)acc;
          acc >>= 32;
          nb -= 32;
        }
      }
    }
  } else {
    if constexpr (BITS == 16) {
#pragma unroll
      for (int i = 0; i < 16; ++i) w[i] = reinterpret_cast<const uint32_t*>(cpos)[i];
    } else {
      int code[32];
      unsigned long long acc = 0;
      int nb = 0, wi = 0;
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        if (nb < BITS) {
          acc |= (unsigned long long)reinterpret_cast<const uint32_t*>(cpos)[wi++] << nb;
          nb += 32;
        }
        code[i] = (int)(acc & ((1u << BITS) - 1));
        acc >>= BITS;
        nb -= BITS;
      }
      pack_slice<BITS>(code, w);
    }
#pragma unroll
    for (int i = 0; i < NW; ++i) *reinterpret_cast<uint32_t*>(tpos + slice_word_offset<BITS>(r, q, i)) = w[i];
  }
  if (BITS < 16 && q == 0) {
    const size_t ci = row * ng + g;
    __half* ts = reinterpret_cast<__half*>(tpos + tile_scale_offset(BITS, r));
    __half* tz = reinterpret_cast<__half*>(tpos + tile_zp_offset(BITS, r));
    if constexpr (EXPORT) {
      can_scales[ci] = *ts;
      can_zps[ci] = *tz;
    } else {
      *ts = can_scales[ci];
      *tz = can_zps[ci];
    }
  }
}

static bool bits_ok(int b) { return b == 16 || b == 8 || b == 4 || b == 3 || b == 2; }
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// A TILED page is one buffer (codes, scales and zero-points of a tile stored together); a CANONICAL page
// below 16 bits has three.
static pw_status check_page_buffers(const pw_page* p, int bits, int layout) {
  if (!p->codes) return PW_ERR_INVALID_ARG;
  if (!aligned16(p->codes)) return PW_ERR_ALIGN;
  if (bits < 16 && layout == PW_LAYOUT_CANONICAL) {
    if (!p->scales || !p->zps) return PW_ERR_INVALID_ARG;
    if (!aligned16(p->scales) || !aligned16(p->zps)) return PW_ERR_ALIGN;
  }
  return PW_OK;
}

// 16-bit sources take two tiles per CTA when the block has an even number of groups.
template <int SK, int SB, int DB>
static void launch_quant(dim3 grid, cudaStream_t s, const void* sc, uint32_t cols, pw_page* d) {
  if (SB == 16 && DB < 16 && grid.x % 2 == 0)
    quant_tile_kernel<SK, SB, DB, (SB == 16 && DB < 16 ? 2 : 1)><<<dim3(grid.x / 2, grid.y), 512, 0, s>>>(sc, cols, d->codes);
  else
    quant_tile_kernel<SK, SB, DB, 1><<<grid, 512, 0, s>>>(sc, cols, d->codes);
}

template <int DB>
static void launch_requant_from4(dim3 grid, cudaStream_t s, const void* sc, pw_page* d) {
  const uint32_t n_tiles = grid.x * grid.y, per_cta = kRequantThreads / kTileRows;
  requant_from4_kernel<DB><<<(n_tiles + per_cta - 1) / per_cta, kRequantThreads, 0, s>>>(sc, n_tiles, d->codes);
}

template <int SK, int SB>
static void launch_quant_dst(int dst_bits, dim3 grid, cudaStream_t s, const void* sc, uint32_t cols, pw_page* d) {
  switch (dst_bits) {
    case 16:
      if (SK == SRC_RAW) launch_quant<SK, SB, 16>(grid, s, sc, cols, d);
      break;
    case 8:
      if (SB > 8) launch_quant<SK, SB, (SB > 8 ? 8 : 2)>(grid, s, sc, cols, d);
      break;
    case 4:
      if (SB > 4) launch_quant<SK, SB, (SB > 4 ? 4 : 2)>(grid, s, sc, cols, d);
      break;
    case 3:
      if (SK == SRC_TILED && SB == 4) launch_requant_from4<3>(grid, s, sc, d);
      else if (SB > 3) launch_quant<SK, SB, (SB > 3 ? 3 : 2)>(grid, s, sc, cols, d);
      break;
    case 2:
      if (SK == SRC_TILED && SB == 4) launch_requant_from4<2>(grid, s, sc, d);
      else launch_quant<SK, SB, 2>(grid, s, sc, cols, d);
      break;
  }
}

}  // namespace pw

using namespace pw;

extern "C" size_t pw_page_bytes(uint32_t rows, uint32_t cols, int bits, int group, size_t* codes_b, size_t* scales_b,
                                size_t* zps_b) {
  if (!bits_ok(bits) || group != kGroup || rows == 0 || cols == 0 || cols % kGroup != 0) return 0;
  const size_t n = (size_t)rows * cols;
  const size_t cb = bits == 16 ? 2 * n : n * (size_t)bits / 8;
  const size_t sb = bits == 16 ? 0 : 2 * (n / kGroup);
  if (codes_b) *codes_b = cb;
  if (scales_b) *scales_b = sb;
  if (zps_b) *zps_b = sb;
  return cb + 2 * sb;
}

extern "C" pw_status pw_quantize_block(pw_ctx* ctx, const void* w, uint32_t rows, uint32_t cols, int bits, pw_page* dst,
                                       pw_stream stream) {
  if (!ctx || !w || !dst) return PW_ERR_INVALID_ARG;
  if (!bits_ok(bits)) return PW_ERR_BITS;
  if (rows == 0 || cols == 0 || rows % kTileRows != 0 || cols % kGroup != 0) return PW_ERR_SHAPE;
  if (!aligned16(w)) return PW_ERR_ALIGN;
  pw_status st = check_page_buffers(dst, bits, PW_LAYOUT_TILED);
  if (st != PW_OK) return st;
  dst->rows = rows;
  dst->cols = cols;
  dst->group = kGroup;
  dst->bits = (uint8_t)bits;
  dst->layout = PW_LAYOUT_TILED;
  dim3 grid(cols / kGroup, rows / kTileRows);
  launch_quant_dst<SRC_RAW, 16>(bits, grid, stream, w, cols, dst);
  ctx->launches++;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

extern "C" pw_status pw_demote_block(pw_ctx* ctx, const pw_page* src, int dst_bits, pw_page* dst, pw_stream stream) {
  if (!ctx || !src || !dst) return PW_ERR_INVALID_ARG;
  if (!bits_ok(src->bits) || !bits_ok(dst_bits) || dst_bits >= src->bits) return PW_ERR_BITS;
  if (src->layout != PW_LAYOUT_TILED) return PW_ERR_STATE;
  if (src->rows == 0 || src->cols == 0 || src->rows % kTileRows != 0 || src->cols % kGroup != 0 ||
      src->group != kGroup)
    return PW_ERR_SHAPE;
  pw_status st = check_page_buffers(src, src->bits, PW_LAYOUT_TILED);
  if (st != PW_OK) return st;
  st = check_page_buffers(dst, dst_bits, PW_LAYOUT_TILED);
  if (st != PW_OK) return st;
  if (dst->codes == src->codes) return PW_ERR_INVALID_ARG;  // a demote is out of place
  dst->rows = src->rows;
  dst->cols = src->cols;
  dst->group = kGroup;
  dst->bits = (uint8_t)dst_bits;
  dst->layout = PW_LAYOUT_TILED;
  dim3 grid(src->cols / kGroup, src->rows / kTileRows);
  switch (src->bits) {
    case 16: launch_quant_dst<SRC_TILED, 16>(dst_bits, grid, stream, src->codes, src->cols, dst); break;
    case 8: launch_quant_dst<SRC_TILED, 8>(dst_bits, grid, stream, src->codes, src->cols, dst); break;
    case 4: launch_quant_dst<SRC_TILED, 4>(dst_bits, grid, stream, src->codes, src->cols, dst); break;
    case 3: launch_quant_dst<SRC_TILED, 3>(dst_bits, grid, stream, src->codes, src->cols, dst); break;
  }
  ctx->launches++;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

template <bool EXPORT>
static pw_status relayout(pw_ctx* ctx, const pw_page* src, pw_page* dst, cudaStream_t stream) {
  if (!ctx || !src || !dst) return PW_ERR_INVALID_ARG;
  if (!bits_ok(src->bits)) return PW_ERR_BITS;
  if (src->layout != (EXPORT ? PW_LAYOUT_TILED : PW_LAYOUT_CANONICAL)) return PW_ERR_STATE;
  if (src->rows == 0 || src->cols == 0 || src->rows % kTileRows != 0 || src->cols % kGroup != 0 ||
      src->group != kGroup)
    return PW_ERR_SHAPE;
  pw_status st = check_page_buffers(src, src->bits, src->layout);
  if (st != PW_OK) return st;
  st = check_page_buffers(dst, src->bits, EXPORT ? PW_LAYOUT_CANONICAL : PW_LAYOUT_TILED);
  if (st != PW_OK) return st;
  if (dst->codes == src->codes) return PW_ERR_INVALID_ARG;
  dst->rows = src->rows;
  dst->cols = src->cols;
  dst->group = kGroup;
  dst->bits = src->bits;
  dst->layout = EXPORT ? PW_LAYOUT_CANONICAL : PW_LAYOUT_TILED;
  dim3 grid(src->cols / kGroup, src->rows / kTileRows);
  // scales / zero-points of the canonical side (read on import, written on export)
  const pw_page* can = EXPORT ? dst : src;
  __half* cs = reinterpret_cast<__half*>(can->scales);
  __half* cz = reinterpret_cast<__half*>(can->zps);
  switch (src->bits) {
    case 16: relayout_kernel<16, EXPORT><<<grid, 512, 0, stream>>>(src->codes, src->cols, dst->codes, cs, cz); break;
    case 8: relayout_kernel<8, EXPORT><<<grid, 512, 0, stream>>>(src->codes, src->cols, dst->codes, cs, cz); break;
    case 4: relayout_kernel<4, EXPORT><<<grid, 512, 0, stream>>>(src->codes, src->cols, dst->codes, cs, cz); break;
    case 3: relayout_kernel<3, EXPORT><<<grid, 512, 0, stream>>>(src->codes, src->cols, dst->codes, cs, cz); break;
    case 2: relayout_kernel<2, EXPORT><<<grid, 512, 0, stream>>>(src->codes, src->cols, dst->codes, cs, cz); break;
  }
  ctx->launches++;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

extern "C" pw_status pw_export_page(pw_ctx* ctx, const pw_page* src, pw_page* dst, pw_stream stream) {
  return relayout<true>(ctx, src, dst, stream);
}
extern "C" pw_status pw_import_page(pw_ctx* ctx, const pw_page* src, pw_page* dst, pw_stream stream) {
  return relayout<false>(ctx, src, dst, stream);
}
