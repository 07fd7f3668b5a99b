// The TILED page layout and the bit-level packing of codes inside it.
//
// A page of `rows x cols` at `bits` is cut into tiles of 128 rows x one group (128 columns).
// Tile (rt, g) is one contiguous image at byte offset (rt * n_groups + g) * tile_bytes(bits) of the
// page buffer: bits * 2048 bytes of codes, then (below 16 bits) the 128 fp16 scales of its rows and
// the 128 fp16 zero-points, so that a forward kernel fetches everything it needs of a tile with one
// bulk copy.  A row of a tile owns bits * 16 bytes = `bits` units of 16 bytes; unit j of row r
// sits at ((j * 128) + r) * 16 inside the tile, so that the 128 threads of a row-per-thread kernel
// read unit j with one contiguous 2 KB access.
//
// Inside a row's units the 128 codes are ordered for cheap unpacking to half2 pairs
// (k, k+1), k even:
//   16 bits: unit j = fp16 weights k = 8j .. 8j+7.
//    8 bits: unit j = codes k = 16j .. 16j+15, one per byte, natural order.
//    4 bits: unit j = codes k = 32j .. 32j+31; word w of it = k0 = 32j + 8w; nibble m (m < 4) holds
//            k0 + 2m, nibble 4+m holds k0 + 2m + 1.
//    2 bits: unit j = codes k = 64j .. 64j+63; word w = k0 = 64j + 16w; field m (m < 8) holds
//            k0 + 2m, field 8+m holds k0 + 2m + 1.
//    3 bits: units 0, 1 = the low two bits of every code in the 2-bit arrangement; unit 2 = the high
//            bits: word w = k0 = 32w; bit m (m < 16) holds k0 + 2m, bit 16+m holds k0 + 2m + 1.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

namespace pw {

__host__ __device__ inline size_t tile_code_bytes(int bits) { return (size_t)bits * 2048; }
// bytes of a whole tile image: codes, then the scales and zero-points of its 128 rows
__host__ __device__ inline size_t tile_bytes(int bits) { return (size_t)bits * 2048 + (bits < 16 ? 512 : 0); }
// scale / zero-point of row r inside a tile image
__host__ __device__ inline size_t tile_scale_offset(int bits, int r) { return (size_t)bits * 2048 + 2 * (size_t)r; }
__host__ __device__ inline size_t tile_zp_offset(int bits, int r) { return (size_t)bits * 2048 + 256 + 2 * (size_t)r; }

// ---- integer codes of a 32-weight slice (quarter of a row-group) -----------------------------
// Slice q (0..3) of a row covers k = 32q .. 32q+31.  Word addresses inside a tile image:
//   8 bits: units 2q, 2q+1 (8 words)   4 bits: unit q (4 words)
//   2 bits: unit q/2, words 2(q%2), 2(q%2)+1          3 bits: that, plus unit 2 word q.
template <int BITS>
struct SliceWords {
  static constexpr int kWords = BITS == 16 ? 16 : BITS == 8 ? 8 : BITS == 4 ? 4 : BITS == 3 ? 3 : 2;
};

// byte offset, inside a tile, of word `i` of slice q of row r
template <int BITS>
__host__ __device__ inline int slice_word_offset(int r, int q, int i) {
  if constexpr (BITS == 16) return ((4 * q + (i >> 2)) * 128 + r) * 16 + (i & 3) * 4;
  if constexpr (BITS == 8) return ((2 * q + (i >> 2)) * 128 + r) * 16 + (i & 3) * 4;
  if constexpr (BITS == 4) return (q * 128 + r) * 16 + i * 4;
  if constexpr (BITS == 2) return ((q >> 1) * 128 + r) * 16 + (2 * (q & 1) + i) * 4;
  // BITS == 3: i = 0, 1 low-plane words, i = 2 high-plane word
  if (i < 2) return ((q >> 1) * 128 + r) * 16 + (2 * (q & 1) + i) * 4;
  return (2 * 128 + r) * 16 + q * 4;
}

// Where the single-bit plane of a 32-weight slice (the third bit of a 3-bit page, the planes of a bit-plane block)
// keeps the bit of pair P = weights (2P, 2P + 1), in the low half-word for the even and in the high half-word for
// the odd weight.  The eight pairs that share a word of 2-bit fields take eight consecutive bits: the four whose
// fields are read in place at the even bits, the four read after the shift by 8 at the odd bits between -- one
// shift of the plane word then moves the bits of four pairs to where the decoder merges them.
__host__ __device__ constexpr int plane_bit_pos(int P) { return 8 * (P >> 3) + 2 * (P & 3) + ((P >> 2) & 1); }

template <int BITS>
__device__ inline void unpack_slice(const uint32_t* w, int (&code)[32]) {
  if constexpr (BITS == 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) code[4 * i + j] = (w[i] >> (8 * j)) & 0xff;
  } else if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        code[8 * i + 2 * m] = (w[i] >> (4 * m)) & 0xf;
        code[8 * i + 2 * m + 1] = (w[i] >> (16 + 4 * m)) & 0xf;
      }
  } else {  // 2 or 3
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        code[16 * i + 2 * m] = (w[i] >> (2 * m)) & 3;
        code[16 * i + 2 * m + 1] = (w[i] >> (16 + 2 * m)) & 3;
      }
    if constexpr (BITS == 3) {
#pragma unroll
      for (int m = 0; m < 16; ++m) {
        code[2 * m] |= ((w[2] >> plane_bit_pos(m)) & 1) << 2;
        code[2 * m + 1] |= ((w[2] >> (16 + plane_bit_pos(m))) & 1) << 2;
      }
    }
  }
}

// Two signed integers saturated to BITS-bit unsigned codes and packed, a above b, under the low bits of c moved
// up by 2 * BITS: one instruction clamps and packs two codes.
template <int BITS>
__device__ __forceinline__ uint32_t pack2_sat(int a, int b, uint32_t c) {
  uint32_t d;
  if constexpr (BITS == 8) asm("cvt.pack.sat.u8.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  else if constexpr (BITS == 4) asm("cvt.pack.sat.u4.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  else asm("cvt.pack.sat.u2.s32.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// pack_slice for codes that have not been clamped from above yet (8, 4 or 2 bits): the same words, built from the
// top of each word down with the saturating pack.
template <int BITS>
__device__ inline void pack_slice_sat(const int (&code)[32], uint32_t* w) {
  if constexpr (BITS == 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      w[i] = pack2_sat<8>(code[4 * i + 1], code[4 * i], pack2_sat<8>(code[4 * i + 3], code[4 * i + 2], 0u));
  } else if constexpr (BITS == 4) {
    // low half-word: the even codes of the word's eight, four bits each; high half-word: the odd ones
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int* c = code + 8 * i;
      uint32_t v = pack2_sat<4>(c[7], c[5], 0u);
      v = pack2_sat<4>(c[3], c[1], v);
      v = pack2_sat<4>(c[6], c[4], v);
      w[i] = pack2_sat<4>(c[2], c[0], v);
    }
  } else {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int* c = code + 16 * i;
      uint32_t v = 0;
#pragma unroll
      for (int m = 3; m >= 0; --m) v = pack2_sat<2>(c[4 * m + 3], c[4 * m + 1], v);   // odd codes, from the top
#pragma unroll
      for (int m = 3; m >= 0; --m) v = pack2_sat<2>(c[4 * m + 2], c[4 * m], v);       // even codes below them
      w[i] = v;
    }
  }
}

template <int BITS>
__device__ inline void pack_slice(const int (&code)[32], uint32_t* w) {
  if constexpr (BITS == 8) {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      uint32_t v = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) v |= (uint32_t)code[4 * i + j] << (8 * j);
      w[i] = v;
    }
  } else if constexpr (BITS == 4) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t v = 0;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        v |= (uint32_t)code[8 * i + 2 * m] << (4 * m);
        v |= (uint32_t)code[8 * i + 2 * m + 1] << (16 + 4 * m);
      }
      w[i] = v;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      uint32_t v = 0;
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        v |= (uint32_t)(code[16 * i + 2 * m] & 3) << (2 * m);
        v |= (uint32_t)(code[16 * i + 2 * m + 1] & 3) << (16 + 2 * m);
      }
      w[i] = v;
    }
    if constexpr (BITS == 3) {
      uint32_t v = 0;
#pragma unroll
      for (int m = 0; m < 16; ++m) {
        v |= (uint32_t)((code[2 * m] >> 2) & 1) << plane_bit_pos(m);
        v |= (uint32_t)((code[2 * m + 1] >> 2) & 1) << (16 + plane_bit_pos(m));
      }
      w[2] = v;
    }
  }
}

// ---- fast unpack of a whole row-group to half2 pairs (forward kernels) -------------------------
// out[p] = (weight k = 2p, weight k = 2p + 1), p = 0 .. 63.  `u` are the row's units in order.
// code -> fp16 via the 0x6400 (= 1024.0) mantissa trick, then one HFMA2 with (scale, zero-point).
__device__ inline __half2 u32_as_h2(uint32_t x) { return *reinterpret_cast<__half2*>(&x); }

__device__ inline __half2 dq_pair(uint32_t magic_or_code, __half2 s2, __half2 z2) {
  const __half2 k1024 = u32_as_h2(0x64006400u);
  return __hfma2(__hsub2(u32_as_h2(magic_or_code), k1024), s2, z2);
}

// the same with the bias to subtract given as a half2 bit pattern (the constant whose mantissa carried the code)
__device__ inline __half2 dq_pair_k(uint32_t biased, uint32_t bias, __half2 s2, __half2 z2) {
  return __hfma2(__hsub2(u32_as_h2(biased), u32_as_h2(bias)), s2, z2);
}

// (a & b) | c as ONE instruction.  Written out because the compiler, given two immediates, emits an AND and an
// OR; with the constants in registers the three-input logic unit does both.
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}
// fp16 constant whose mantissa reads a field that starts at bit POS as an integer: 2^(10 - POS) has its unit in
// the last place at bit POS, so (field << POS) | bits(2^(10 - POS)) = 2^(10 - POS) + field, exactly.
template <int POS>
__device__ __forceinline__ constexpr uint32_t field_magic() {
  return (uint32_t)((25 - POS) << 10) * 0x00010001u;
}
// The pair of W-bit fields at bit POS of the two half-words of `word` -> (field * scale + zero-point) as half2.
template <int POS, int W>
__device__ __forceinline__ __half2 dq_field(uint32_t word, __half2 s2, __half2 z2) {
  constexpr uint32_t mask = (((1u << W) - 1u) << POS) * 0x00010001u;
  constexpr uint32_t magic = field_magic<POS>();
  return dq_pair_k(and_or(word, mask, magic), magic, s2, z2);
}
// The same for a 2-bit field, with (BITS == 3) the code's third bit, already moved to bit POS + 2 of `hi`, put just
// above it.
template <int POS, int BITS>
__device__ __forceinline__ __half2 dq_field23(uint32_t word, uint32_t hi, __half2 s2, __half2 z2) {
  constexpr uint32_t mask = (3u << POS) * 0x00010001u;
  constexpr uint32_t magic = field_magic<POS>();
  uint32_t v = and_or(word, mask, magic);
  if constexpr (BITS == 3) v = and_or(hi, (1u << (POS + 2)) * 0x00010001u, v);
  return dq_pair_k(v, magic, s2, z2);
}

// Quarter t (0 .. 3) of a row-group: out[p] = weights (32t + 2p, 32t + 2p + 1), p = 0 .. 15.
// `row_units` points at unit 0 of the row inside a tile image (shared or global memory); unit j
// of the same row is kUnitStride uint4 further on.
constexpr int kUnitStride = 128;  // uint4 elements between consecutive units of one row

template <int BITS>
__device__ __forceinline__ void decode_quarter(const uint4* row_units, int t, __half2 s2, __half2 z2, __half2* out) {
  if constexpr (BITS == 16) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint4 u = row_units[(4 * t + j) * kUnitStride];
      out[4 * j + 0] = u32_as_h2(u.x);
      out[4 * j + 1] = u32_as_h2(u.y);
      out[4 * j + 2] = u32_as_h2(u.z);
      out[4 * j + 3] = u32_as_h2(u.w);
    }
  } else if constexpr (BITS == 8) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const uint4 u = row_units[(2 * t + j) * kUnitStride];
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        out[8 * j + 2 * i] = dq_pair(__byte_perm(w[i], 0x64646464u, 0x4140), s2, z2);
        out[8 * j + 2 * i + 1] = dq_pair(__byte_perm(w[i], 0x64646464u, 0x4342), s2, z2);
      }
    }
  } else if constexpr (BITS == 4) {
    // A nibble at mantissa bits 0-3 of 0x6400 reads 1024 + code; at bits 4-7 of 0x5400 it reads 64 + code.  One
    // shift by 8 per word brings the other two nibbles of each half-word to those positions.
    const uint4 u = row_units[t * kUnitStride];
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t w8 = w[i] >> 8;
      out[4 * i + 0] = dq_field<0, 4>(w[i], s2, z2);
      out[4 * i + 1] = dq_field<4, 4>(w[i], s2, z2);
      out[4 * i + 2] = dq_field<0, 4>(w8, s2, z2);
      out[4 * i + 3] = dq_field<4, 4>(w8, s2, z2);
    }
  } else {
    // 2 bits: words 2(t%2), 2(t%2)+1 of unit t/2.  3 bits: the same low-plane words plus word t of unit 2.
    // A half-word holds eight 2-bit fields; fields 0 .. 3 are read where they lie (see dq_field), one shift by 8
    // per word brings fields 4 .. 7 to the same places.  The third bit of a 3-bit code is moved to the place
    // just above its field, where it reads 4: the plane word keeps the bits of fields 0 .. 3 of word i at bits
    // 8i, 8i + 2, .. and those of fields 4 .. 7 at the odd bits between (plane_bit_pos), so two shifts per word do.
    const uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint32_t*>(row_units + (t >> 1) * kUnitStride) +
                                                     2 * (t & 1));
    const uint32_t w[2] = {u.x, u.y};
    uint32_t hw = 0;
    if constexpr (BITS == 3) hw = reinterpret_cast<const uint32_t*>(row_units + 2 * kUnitStride)[t];
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const uint32_t w8 = w[i] >> 8;
      // third bits of fields 0 .. 3 / 4 .. 7 at bits 2(m mod 4) + 2
      const uint32_t ha = i == 0 ? hw << 2 : hw >> 6, hb = i == 0 ? hw << 1 : hw >> 7;
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        const int p = 8 * i + m;                   // pair index inside the quarter
        const uint32_t src = m < 4 ? w[i] : w8, hi = m < 4 ? ha : hb;
        switch (m & 3) {
          case 0: out[p] = dq_field23<0, BITS>(src, hi, s2, z2); break;
          case 1: out[p] = dq_field23<2, BITS>(src, hi, s2, z2); break;
          case 2: out[p] = dq_field23<4, BITS>(src, hi, s2, z2); break;
          default: out[p] = dq_field23<6, BITS>(src, hi, s2, z2); break;
        }
      }
    }
  }
}

// Half h (0 or 1) of a row-group: out[p] = weights (64h + 2p, 64h + 2p + 1), p = 0 .. 31.
template <int BITS>
__device__ __forceinline__ void decode_half(const uint4* row_units, int h, __half2 s2, __half2 z2, __half2* out) {
  decode_quarter<BITS>(row_units, 2 * h, s2, z2, out);
  decode_quarter<BITS>(row_units, 2 * h + 1, s2, z2, out + 16);
}

// ---- overlaid bit-plane pages (PW_LAYOUT_PLANES) -----------------------------------------------
// A block quantized once to a 4-bit master code c4 is stored as three plane buffers, each cut into the same
// (128-row, one-group) tiles as a TILED page: tile (rt, g) of a plane is one contiguous image at
// (rt * n_groups + g) * tile size.
//   TOP   5632 B per tile: the two leading bits of every code in the 2-bit arrangement above (4096 B), then the
//         lookup-table state of each bitwidth the planes can be read at: 128 scales + 128 zero-points (fp16) for
//         2 bits, the same for 3 bits, the same for 4 bits.  The table is affine, entry c = zero-point + c * scale.
//   BIT1  2048 B per tile: the third bit.  Row r owns 16 bytes at r * 16; word w of them covers k = 32w .. 32w+31,
//         the even k in its low half-word, the odd k in its high half-word, pair P = (k = 32w + 2P, 32w + 2P + 1)
//         at bit plane_bit_pos(P) of each: the eight pairs that share a word of top codes take eight consecutive
//         bits, first the four whose top codes are read in place (at every other bit), then, in the bits between,
//         the four whose top codes are read after a shift by 8 -- so that one shift of the plane word puts the
//         bits of four pairs where the decoder wants them (see decode_quarter_planes).
//   BIT0  the fourth bit, same arrangement.
// Read at q bits the code of a weight is its first q bits, c4 >> (4 - q): q = 2 needs TOP alone, q = 3 TOP and
// BIT1, q = 4 all three.  Lowering the precision moves and computes nothing.
constexpr int kPlaneTopCodes = 4096;
constexpr int kPlaneTopTile = kPlaneTopCodes + 3 * 512;
constexpr int kPlaneBitTile = 2048;
__host__ __device__ inline int plane_lut_offset(int q) { return kPlaneTopCodes + 512 * (q - 2); }
// image of one tile inside a ring slot of the FFN kernels: top codes, BIT1, BIT0, then the table state of the
// committed bitwidth (fixed offsets whatever the bitwidth)
constexpr int kPlaneSlotBit1 = 4096, kPlaneSlotBit0 = 6144, kPlaneSlotLut = 8192;
constexpr int kPlaneSlotBytes = kPlaneSlotLut + 512;

// Quarter t of a row-group read from such an image at Q = 3 or 4 bits (Q = 2 is the plain 2-bit decoder on the
// top codes): out[p] = weights (32t + 2p, 32t + 2p + 1).
template <int Q>
__device__ __forceinline__ void decode_quarter_planes(const char* image, int r, int t, __half2 s2, __half2 z2, __half2* out) {
  const uint4* row_units = reinterpret_cast<const uint4*>(image) + r;
  const uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<const uint32_t*>(row_units + (t >> 1) * kUnitStride) +
                                                   2 * (t & 1));
  const uint32_t w[2] = {u.x, u.y};
  const uint32_t h1 = reinterpret_cast<const uint32_t*>(image + kPlaneSlotBit1 + r * 16)[t];
  uint32_t h0 = 0;
  if constexpr (Q == 4) h0 = reinterpret_cast<const uint32_t*>(image + kPlaneSlotBit0 + r * 16)[t];
  // The top two bits of pair m of a word sit at bit 2m of both half-words.  Shifted up by Q - 2 places they stand
  // where the leading bits of a Q-bit code belong when the unit of the fp16 constant is at bit 2(m mod 4) (see
  // dq_field).  The plane bits below them: pairs 0 .. 3 of word i have theirs at bits 8i, 8i + 2, 8i + 4, 8i + 6 of
  // the plane word, pairs 4 .. 7 at the odd bits between, so one shift per word, plane and group of four pairs
  // moves four of them to their places at once, and one logic instruction each merges them.
  constexpr int up = Q - 2;
  auto moved = [](uint32_t x, int s) { return s >= 0 ? x >> s : x << -s; };   // s is a constant after unrolling
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const uint32_t lo4 = w[i] << up, hi4 = w[i] >> (8 - up);   // pairs 0 .. 3 / 4 .. 7 of the word at bits up + 2(m mod 4)
    // plane bits of pairs 0 .. 3 / 4 .. 7 at bits 2(m mod 4) + up - 1 (third bit) and 2(m mod 4) (fourth bit)
    uint32_t a1 = moved(h1, 8 * i - (up - 1)), b1 = moved(h1, 8 * i + 1 - (up - 1));
    if constexpr (Q == 4) {
      // third and fourth bits of four pairs side by side (bits 2(m mod 4) + 1 and 2(m mod 4)): merged once per four
      // pairs, so that a pair takes its two low bits with one instruction
      a1 = and_or(a1, 0x00aa00aau, (h0 >> (8 * i)) & 0x00550055u);
      b1 = and_or(b1, 0x00aa00aau, (h0 >> (8 * i + 1)) & 0x00550055u);
    }
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      const int p = 8 * i + m;                     // pair index inside the quarter
      const int U = 2 * (m & 3);                   // where the code's last bit goes
      const uint32_t magic = (uint32_t)((25 - U) << 10) * 0x00010001u;
      uint32_t v = and_or(m < 4 ? lo4 : hi4, (3u << (U + up)) * 0x00010001u, magic);
      v = and_or(m < 4 ? a1 : b1, (Q == 4 ? 3u << U : 1u << U) * 0x00010001u, v);
      out[p] = dq_pair_k(v, magic, s2, z2);
    }
  }
}
template <int Q>
__device__ __forceinline__ void decode_half_planes(const char* image, int r, int h, __half2 s2, __half2 z2, __half2* out) {
  if constexpr (Q == 2) {
    decode_half<2>(reinterpret_cast<const uint4*>(image) + r, h, s2, z2, out);
  } else {
    decode_quarter_planes<Q>(image, r, 2 * h, s2, z2, out);
    decode_quarter_planes<Q>(image, r, 2 * h + 1, s2, z2, out + 16);
  }
}

}  // namespace pw
