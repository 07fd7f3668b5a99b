// Oracle for the paged-weight MoE hot path.  TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, single-translation-unit CPU statement of what the GPU library
// computes.  Only the tests, the smoke check and the benchmark's CPU-baseline
// leg may load it; the product path never does, and it shares no code, tables
// or helpers with the CUDA sources.
//
// What it follows (paper passages):
//   * top-K routing of E experts per token                     (Sec. 2.1)
//   * one linear-block = one weight matrix of one expert, each with its own
//     committed bitwidth q_i read from a page-table row         (Sec. 3.1)
//   * size table M_i^b and released bytes M^b - M^b'            (Eq. 3)
//   * routing, expert activation, down projection and output
//     accumulation of the mixed-precision MoE layer             (Sec. 3.3)
//   * offload = lower the committed bitwidth of a block         (Sec. 3.1, 3.3)
// The paper stores Any-Precision bit-planes with a centroid table whose
// construction it does not give; this build's pages are group-wise uniform
// integer codes (group 128 along the input dimension, fp16 scale, fp16
// zero-point = the value code 0 decodes to).  Parity against the authors'
// implementation is therefore unpinned; every function below is pinned by the
// invariants and closed forms in tests/test_oracle_*.py.
//
// Arithmetic rules: quantization is fp32, one IEEE round-to-nearest-even per
// operation, in the order written (compile with -ffp-contract=off, no
// fast-math).  Forward dot products accumulate in double over ascending index
// and are stored as fp32; SwiGLU and the gate-weighted combine are fp32.
//
// Build: g++ -O2 -std=c++17 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC

#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <vector>
#include <algorithm>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---- fp16 <-> fp32, written out (no hardware half type) -------------------
float h2f(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  uint32_t exp = (h >> 10) & 0x1fu;
  uint32_t man = h & 0x3ffu;
  uint32_t bits;
  if (exp == 0) {
    if (man == 0) {
      bits = sign;
    } else {  // subnormal: value = man * 2^-24
      float v = (float)man * 5.9604644775390625e-08f;
      std::memcpy(&bits, &v, 4);
      bits |= sign;
    }
  } else if (exp == 31) {
    bits = sign | 0x7f800000u | (man << 13);
  } else {
    bits = sign | ((exp + 112u) << 23) | (man << 13);
  }
  float f;
  std::memcpy(&f, &bits, 4);
  return f;
}

// round-to-nearest-even fp32 -> fp16
uint16_t f2h(float f) {
  uint32_t x;
  std::memcpy(&x, &f, 4);
  uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  uint32_t ax = x & 0x7fffffffu;
  if (ax >= 0x7f800000u) {  // inf / nan
    return (uint16_t)(sign | 0x7c00u | ((ax > 0x7f800000u) ? 0x200u : 0u));
  }
  if (ax >= 0x477ff000u) {  // >= 65520 rounds to inf
    return (uint16_t)(sign | 0x7c00u);
  }
  if (ax < 0x33000001u) {  // <= 2^-25 rounds to zero (tie at 2^-25 goes to even = 0)
    return sign;
  }
  int e = (int)(ax >> 23) - 127;
  uint32_t m = (ax & 0x7fffffu) | 0x800000u;  // 24-bit significand
  int shift;                                    // bits dropped from m
  uint32_t base;
  if (e < -14) {  // subnormal result: value = q * 2^-24
    shift = 13 + (-14 - e);
    base = 0;
  } else {
    shift = 13;
    base = (uint32_t)(e + 15) << 10;
    m &= 0x7fffffu;
  }
  uint32_t q = m >> shift;
  uint32_t rem = m & ((1u << shift) - 1u);
  uint32_t half = 1u << (shift - 1);
  if (rem > half || (rem == half && (q & 1u))) q += 1;  // carry may bump the exponent: correct
  return (uint16_t)(sign | (base + q));
}

inline int levels(int bits) { return (1 << bits) - 1; }

inline bool bits_ok(int bits) { return bits == 16 || bits == 8 || bits == 4 || bits == 3 || bits == 2; }

// Canonical packed layout: code of element n = r*cols + c sits at stream bits
// [n*b, (n+1)*b), stream bit j = bit (j & 7) of byte (j >> 3).
inline void put_code(uint8_t* codes, size_t n, int b, uint32_t code) {
  size_t bit = n * (size_t)b;
  for (int i = 0; i < b; ++i, ++bit) {
    if ((code >> i) & 1u) codes[bit >> 3] |= (uint8_t)(1u << (bit & 7));
  }
}
inline uint32_t get_code(const uint8_t* codes, size_t n, int b) {
  size_t bit = n * (size_t)b;
  uint32_t code = 0;
  for (int i = 0; i < b; ++i, ++bit) {
    code |= (uint32_t)((codes[bit >> 3] >> (bit & 7)) & 1u) << i;
  }
  return code;
}

// Group quantizer Q(w, b): one group of `group` fp16 values -> codes, scale, zero-point.
void quantize_group(const uint16_t* w, int group, int b, uint32_t* code_out, uint16_t* scale_h, uint16_t* zp_h) {
  const int L = levels(b);
  float lo = h2f(w[0]), hi = lo;
  for (int i = 1; i < group; ++i) {
    float v = h2f(w[i]);
    if (v < lo) lo = v;
    if (v > hi) hi = v;
  }
  if (lo == 0.0f) lo = 0.0f;  // -0 is stored as +0
  float r = hi - lo;
  uint16_t sh;
  if (r == 0.0f) {
    sh = 0x3c00u;  // 1.0
  } else {
    sh = f2h(r / (float)L);
    if ((sh & 0x7fffu) == 0) sh = 0x0001u;  // smallest fp16 subnormal, 2^-24
  }
  *scale_h = sh;
  *zp_h = f2h(lo);  // exact: lo is one of the fp16 inputs
  float s = h2f(sh);
  float rinv = 1.0f / s;
  for (int i = 0; i < group; ++i) {
    float d = h2f(w[i]) - lo;
    float q = d * rinv;
    float c = rintf(q);  // round-half-even under the default rounding mode
    if (c < 0.0f) c = 0.0f;
    if (c > (float)L) c = (float)L;
    code_out[i] = (uint32_t)c;
  }
}

// D(code, scale, zp): the fp16 weight a stored code stands for.
inline uint16_t dequant_one(uint32_t code, uint16_t scale_h, uint16_t zp_h) {
  float p = (float)code * h2f(scale_h);  // exact in fp32
  float v = p + h2f(zp_h);
  return f2h(v);
}

struct Page {
  const void* codes;
  const uint16_t* scales;
  const uint16_t* zps;
  uint32_t rows, cols;
  int32_t group, bits;
};

// Dequantize a whole page to fp32 values (each one exactly an fp16 number).
void page_to_f32(const Page& pg, std::vector<float>& out) {
  size_t n = (size_t)pg.rows * pg.cols;
  out.resize(n);
  if (pg.bits == 16) {
    const uint16_t* w = (const uint16_t*)pg.codes;
#pragma omp parallel for schedule(static)
    for (long long i = 0; i < (long long)n; ++i) out[i] = h2f(w[i]);
    return;
  }
  const uint8_t* codes = (const uint8_t*)pg.codes;
  size_t ng = pg.cols / pg.group;
#pragma omp parallel for schedule(static)
  for (long long r = 0; r < (long long)pg.rows; ++r) {
    for (size_t g = 0; g < ng; ++g) {
      uint16_t sh = pg.scales[(size_t)r * ng + g], zh = pg.zps[(size_t)r * ng + g];
      for (int i = 0; i < pg.group; ++i) {
        size_t idx = (size_t)r * pg.cols + g * pg.group + i;
        out[idx] = h2f(dequant_one(get_code(codes, idx, pg.bits), sh, zh));
      }
    }
  }
}

}  // namespace

extern "C" {

uint16_t orc_f32_to_f16(float f) { return f2h(f); }
float orc_f16_to_f32(uint16_t h) { return h2f(h); }

// Size table M_i^b (Eq. 3): bytes of a rows x cols block at `bits`, metadata included.
// Returns 0 on an invalid shape or bitwidth.
uint64_t orc_page_bytes(uint32_t rows, uint32_t cols, int bits, int group, uint64_t* codes_b, uint64_t* scales_b,
                        uint64_t* zps_b) {
  if (!bits_ok(bits) || group <= 0 || cols % (uint32_t)group != 0 || rows == 0 || cols == 0) return 0;
  uint64_t n = (uint64_t)rows * cols;
  uint64_t cb, sb;
  if (bits == 16) {
    cb = 2 * n;
    sb = 0;
  } else {
    cb = n * (uint64_t)bits / 8;
    sb = 2 * (n / (uint64_t)group);
  }
  if (codes_b) *codes_b = cb;
  if (scales_b) *scales_b = sb;
  if (zps_b) *zps_b = sb;
  return cb + 2 * sb;
}

// fp16 block [rows, cols] -> b-bit page in the canonical layout.
// bits == 16 copies the weights verbatim into `codes` and leaves scales / zps untouched.
int orc_quantize_block(const uint16_t* w, uint32_t rows, uint32_t cols, int bits, int group, uint8_t* codes,
                       uint16_t* scales, uint16_t* zps) {
  if (!bits_ok(bits) || group <= 0 || cols % (uint32_t)group != 0) return 1;
  size_t n = (size_t)rows * cols;
  if (bits == 16) {
    std::memcpy(codes, w, 2 * n);
    return 0;
  }
  std::memset(codes, 0, n * (size_t)bits / 8);
  size_t ng = cols / group;
#pragma omp parallel for schedule(static)
  for (long long r = 0; r < (long long)rows; ++r) {
    std::vector<uint32_t> tmp(group);
    for (size_t g = 0; g < ng; ++g) {
      uint16_t sh, zh;
      size_t base = (size_t)r * cols + g * group;
      quantize_group(w + base, group, bits, tmp.data(), &sh, &zh);
      scales[(size_t)r * ng + g] = sh;
      zps[(size_t)r * ng + g] = zh;
      // a group is 16*b bytes and starts on a byte boundary, so rows never share a byte
      for (int i = 0; i < group; ++i) put_code(codes, base + i, bits, tmp[i]);
    }
  }
  return 0;
}

// page -> the fp16 tensor it represents.
int orc_dequantize_block(const uint8_t* codes, const uint16_t* scales, const uint16_t* zps, uint32_t rows,
                         uint32_t cols, int bits, int group, uint16_t* w_out) {
  if (!bits_ok(bits) || group <= 0 || cols % (uint32_t)group != 0) return 1;
  size_t n = (size_t)rows * cols;
  if (bits == 16) {
    std::memcpy(w_out, codes, 2 * n);
    return 0;
  }
  size_t ng = cols / group;
#pragma omp parallel for schedule(static)
  for (long long r = 0; r < (long long)rows; ++r) {
    for (size_t g = 0; g < ng; ++g) {
      uint16_t sh = scales[(size_t)r * ng + g], zh = zps[(size_t)r * ng + g];
      for (int i = 0; i < group; ++i) {
        size_t idx = (size_t)r * cols + g * group + i;
        w_out[idx] = dequant_one(get_code(codes, idx, bits), sh, zh);
      }
    }
  }
  return 0;
}

// Demote: Q(D(src page), dst_bits).  The source is not modified.
int orc_demote_block(const uint8_t* src_codes, const uint16_t* src_scales, const uint16_t* src_zps, uint32_t rows,
                     uint32_t cols, int src_bits, int dst_bits, int group, uint8_t* dst_codes, uint16_t* dst_scales,
                     uint16_t* dst_zps) {
  if (!bits_ok(src_bits) || !bits_ok(dst_bits) || dst_bits >= src_bits) return 1;
  std::vector<uint16_t> w((size_t)rows * cols);
  int rc = orc_dequantize_block(src_codes, src_scales, src_zps, rows, cols, src_bits, group, w.data());
  if (rc) return rc;
  return orc_quantize_block(w.data(), rows, cols, dst_bits, group, dst_codes, dst_scales, dst_zps);
}

// Router: per token the k largest logits (ties: lower expert index first), gates =
// softmax over those k logits, summed in slot order.
int orc_router(const float* logits, int T, int E, int k, int32_t* topk_ids, float* gates) {
  if (k < 1 || k > E) return 1;
  std::vector<int> order(E);
  for (int t = 0; t < T; ++t) {
    const float* l = logits + (size_t)t * E;
    for (int e = 0; e < E; ++e) order[e] = e;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return l[a] > l[b]; });
    float l0 = l[order[0]];
    std::vector<float> p(k);
    float S = 0.0f;
    for (int j = 0; j < k; ++j) {
      p[j] = expf(l[order[j]] - l0);
      S = S + p[j];
    }
    for (int j = 0; j < k; ++j) {
      topk_ids[(size_t)t * k + j] = order[j];
      gates[(size_t)t * k + j] = p[j] / S;
    }
  }
  return 0;
}

// Stable counting sort of the T*k (token, slot) pairs by expert.
int orc_permute(const int32_t* topk_ids, int T, int k, int E, int32_t* counts, int32_t* offsets, int32_t* perm,
                int32_t* inv_perm) {
  int P = T * k;
  for (int e = 0; e < E; ++e) counts[e] = 0;
  for (int p = 0; p < P; ++p) {
    if (topk_ids[p] < 0 || topk_ids[p] >= E) return 1;
    counts[topk_ids[p]]++;
  }
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
  std::vector<int32_t> cursor(offsets, offsets + E);
  for (int p = 0; p < P; ++p) {
    int pos = cursor[topk_ids[p]]++;
    perm[pos] = p;
    inv_perm[p] = pos;
  }
  return 0;
}

struct orc_page {  // mirrors Page; pointers are host memory, canonical layout
  const void* codes;
  const uint16_t* scales;
  const uint16_t* zps;
  uint32_t rows, cols;
  int32_t group, bits;
};

// y = W_down( silu(W_gate x) * (W_up x) ) for one token row; Wg, Wu are [F,H], Wd is [H,F].
static void ffn_token(const float* Wg, const float* Wu, const float* Wd, const float* x, int H, int F, float* h,
                      float* y) {
  for (int f = 0; f < F; ++f) {
    const float* wg = Wg + (size_t)f * H;
    const float* wu = Wu + (size_t)f * H;
    double ag = 0.0, au = 0.0;
    for (int c = 0; c < H; ++c) {
      ag += (double)wg[c] * (double)x[c];
      au += (double)wu[c] * (double)x[c];
    }
    float g = (float)ag, u = (float)au;
    float sig = g / (1.0f + expf(-g));
    h[f] = sig * u;
  }
  for (int r = 0; r < H; ++r) {
    const float* wd = Wd + (size_t)r * F;
    double a = 0.0;
    for (int f = 0; f < F; ++f) a += (double)wd[f] * (double)h[f];
    y[r] = (float)a;
  }
}

// Whole layer forward.  `pages` holds (E + n_shared) * 3 entries ordered
// [expert][gate, up, down]; experts E .. E+n_shared-1 are always-on shared experts
// (gate 1, added after the routed sum).  token_mask (may be NULL) selects the
// tokens whose output rows are computed; other rows of `out` are left untouched.
int orc_moe_forward(const uint16_t* hidden, const float* logits, int T, int E, int n_shared, int k, int H, int F,
                    const orc_page* pages, const uint8_t* token_mask, float* out) {
  int P = T * k;
  std::vector<int32_t> ids(P), counts(E), offsets(E + 1), perm(P), inv(P);
  std::vector<float> gates(P);
  if (orc_router(logits, T, E, k, ids.data(), gates.data())) return 1;
  if (orc_permute(ids.data(), T, k, E, counts.data(), offsets.data(), perm.data(), inv.data())) return 1;

  std::vector<float> x((size_t)T * H);
  for (size_t i = 0; i < x.size(); ++i) x[i] = h2f(hidden[i]);

  // y of every routed pair, in permuted (expert-segment) order, then of every shared expert
  std::vector<float> y((size_t)P * H, 0.0f);
  std::vector<float> ysh((size_t)n_shared * T * H, 0.0f);
  std::vector<float> Wg, Wu, Wd;
  for (int e = 0; e < E + n_shared; ++e) {
    bool shared = e >= E;
    std::vector<int> toks, dst;  // token index and destination row of each selected pair
    if (!shared) {
      for (int pos = offsets[e]; pos < offsets[e + 1]; ++pos) {
        int t = perm[pos] / k;
        if (token_mask && !token_mask[t]) continue;
        toks.push_back(t);
        dst.push_back(pos);
      }
    } else {
      for (int t = 0; t < T; ++t) {
        if (token_mask && !token_mask[t]) continue;
        toks.push_back(t);
        dst.push_back(t);
      }
    }
    if (toks.empty()) continue;
    const orc_page* pg = pages + (size_t)e * 3;
    for (int u = 0; u < 3; ++u) {
      if (!bits_ok(pg[u].bits)) return 2;
      uint32_t er = (u == 2) ? (uint32_t)H : (uint32_t)F, ec = (u == 2) ? (uint32_t)F : (uint32_t)H;
      if (pg[u].rows != er || pg[u].cols != ec) return 3;
    }
    Page a{pg[0].codes, pg[0].scales, pg[0].zps, pg[0].rows, pg[0].cols, pg[0].group, pg[0].bits};
    Page b{pg[1].codes, pg[1].scales, pg[1].zps, pg[1].rows, pg[1].cols, pg[1].group, pg[1].bits};
    Page c{pg[2].codes, pg[2].scales, pg[2].zps, pg[2].rows, pg[2].cols, pg[2].group, pg[2].bits};
    page_to_f32(a, Wg);
    page_to_f32(b, Wu);
    page_to_f32(c, Wd);
    float* ybase = shared ? ysh.data() + (size_t)(e - E) * T * H : y.data();
#pragma omp parallel
    {
      std::vector<float> h(F);
#pragma omp for schedule(dynamic, 1)
      for (long long i = 0; i < (long long)toks.size(); ++i) {
        ffn_token(Wg.data(), Wu.data(), Wd.data(), x.data() + (size_t)toks[i] * H, H, F, h.data(),
                  ybase + (size_t)dst[i] * H);
      }
    }
  }
  for (int t = 0; t < T; ++t) {
    if (token_mask && !token_mask[t]) continue;
    float* o = out + (size_t)t * H;
    for (int c = 0; c < H; ++c) o[c] = 0.0f;
    for (int j = 0; j < k; ++j) {
      float gw = gates[(size_t)t * k + j];
      const float* yy = y.data() + (size_t)inv[(size_t)t * k + j] * H;
      for (int c = 0; c < H; ++c) {
        float term = gw * yy[c];
        o[c] = o[c] + term;
      }
    }
    for (int s = 0; s < n_shared; ++s) {
      const float* yy = ysh.data() + ((size_t)s * T + t) * H;
      for (int c = 0; c < H; ++c) o[c] = o[c] + yy[c];
    }
  }
  return 0;
}

// Brute-force cross-check for tiny inputs: every token visits every routed expert,
// unselected experts get gate 0; no permutation, no segments.  Terms are added in
// ascending expert order, so the result equals orc_moe_forward up to fp32 summation order.
int orc_moe_forward_bruteforce(const uint16_t* hidden, const float* logits, int T, int E, int n_shared, int k, int H,
                               int F, const orc_page* pages, float* out) {
  int P = T * k;
  std::vector<int32_t> ids(P);
  std::vector<float> gates(P);
  if (orc_router(logits, T, E, k, ids.data(), gates.data())) return 1;
  std::vector<std::vector<float>> W((size_t)(E + n_shared) * 3);
  for (int e = 0; e < E + n_shared; ++e)
    for (int u = 0; u < 3; ++u) {
      const orc_page& q = pages[(size_t)e * 3 + u];
      Page pg{q.codes, q.scales, q.zps, q.rows, q.cols, q.group, q.bits};
      page_to_f32(pg, W[(size_t)e * 3 + u]);
    }
  std::vector<float> x(H), h(F), yv(H);
  for (int t = 0; t < T; ++t) {
    for (int c = 0; c < H; ++c) x[c] = h2f(hidden[(size_t)t * H + c]);
    float* o = out + (size_t)t * H;
    for (int c = 0; c < H; ++c) o[c] = 0.0f;
    for (int e = 0; e < E + n_shared; ++e) {
      float gw = 0.0f;
      if (e >= E) {
        gw = 1.0f;
      } else {
        for (int j = 0; j < k; ++j)
          if (ids[(size_t)t * k + j] == e) gw = gates[(size_t)t * k + j];
      }
      ffn_token(W[(size_t)e * 3].data(), W[(size_t)e * 3 + 1].data(), W[(size_t)e * 3 + 2].data(), x.data(), H, F,
                h.data(), yv.data());
      for (int c = 0; c < H; ++c) {
        float term = gw * yv[c];
        o[c] = o[c] + term;
      }
    }
  }
  return 0;
}

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
