// Tensor-core expert FFN for sm_100a.
//
//   D[128 weight rows, N tokens] += W[128, 16] * X[N, 16]^T      (tcgen05.mma, kind::f16, fp32 in TMEM)
//
// Weight pages stream HBM -> shared memory with bulk async copies into a ring of 34 KB slots.  What travels
// in one copy is a "chunk": up to four consecutive tile images of one row tile of a quantized page (a tile
// image = 128 rows x one group: codes, scales, zero-points; consecutive groups of a row tile are contiguous
// in the page), two for 8-bit pages, or one whole 16-bit tile (32 KB).  Chunks are numbered in issue order;
// number `seq` lives in slot seq mod n_slots, so every role finds its own chunks from their numbers alone.
// A 16-bit tile is already in the tensor core's K-major core-matrix layout: the MMA reads it from shared
// memory as the A operand without any thread touching it.  A quantized tile is unpacked and dequantized in
// registers (one weight row per thread) and written to tensor memory, which the MMA then reads as its A
// operand.  The token tile (B operand) comes from the k-chunk-major operand buffers with one 2-D TMA copy
// per group.
//
// One persistent CTA per SM, 26 warps.  The arithmetic pipes that the dequantizers use run at half rate and
// are shared with every control instruction, so each role does as little per tile as it can: a unit's
// description is read from global memory once (by the weight producer) and handed to the other roles through
// shared memory, barrier traffic of the ring is per chunk, and the dequantizer loop is compiled once per
// bitwidth with nothing but the decode between its waits.
//   warps 0-15   dequantize: four groups of four warps; tile k of a matrix goes to that matrix's group
//                k mod (groups per matrix); warp w owns TMEM lanes 32*(w%4).., one weight row per thread;
//                a group has one operand slot of 64 columns in tensor memory (a whole tile, K 0..127) and hands
//                it to its issuer once per tile, while it decodes the first half of its next tile in registers;
//   warp 16      weight producer: claims the CTA's units from a global counter, posts their descriptions on the
//                CTA's work list and issues the chunk copies as far ahead as the ring allows;
//   warp 17      token-tile producer (its own few slots, never holds back the weight stream);
//   warps 18-21  MMA issuers (warp 18 also allocates tensor memory).  Dependent MMAs into one accumulator
//                follow each other ~100 cycles apart whatever their size, so the issuers work in parallel:
//                issuer j of a matrix issues all eight k-steps of the tiles k = j mod (issuers per matrix) into
//                its own partial accumulator -- with as many issuers as groups, each dequantizer group has an
//                issuer of its own -- and no two threads ever accumulate into the same columns;
//   warps 22-25  epilogue: adds the partials; SwiGLU -> fp16 operand of the down projection (PHASE 0), or the
//                fp32 split-K partial of the down projection (PHASE 1).  Narrow token tiles alternate
//                between two accumulator buffers, so the next unit's MMAs overlap the epilogue.
//                Token tiles wider than 64 leave no second buffer: the HELP instantiation, launched for
//                those, has the four issuer warps share the epilogue of every wide unit.
// Every wait is bounded; when one runs out the CTA records PW_ERR_TIMEOUT in the status word, stops issuing
// work, frees its tensor memory and returns.
#include <cuda.h>

#include <new>

#include "pw_common.cuh"
#include "pw_layout.cuh"

namespace pw {

constexpr int kSlotBytes = 34816;              // one ring slot: four 4-bit tile images (4 x 8704), two 8-bit, one 16-bit tile
constexpr int kMaxSlots = 6;
constexpr int kChunkArrivals = 16;             // arrivals that hand a slot back: four tiles x four warps
constexpr int kMaxASlots = 4;                  // operand slots in tensor memory, one per group (64 columns = a 128 x 128 tile)
constexpr int kMaxBSlots = 5;
constexpr int kSched = 32;                     // entries of the CTA's work list
constexpr int kCtrlBytes = 2048;
constexpr int kMaxDynSmem = 232448;            // 227 KB
constexpr int kDqWarps = 16;
constexpr int kWarpW = 16, kWarpB = 17, kWarpMma = 18, kIssuers = 4, kWarpEpi = 22;
constexpr int kThreads = 832;
constexpr int kTmemCols = 512;
constexpr uint32_t kSuspendHintNs = 20000;     // a blocked barrier wait sleeps up to this long per poll
constexpr uint32_t kDefaultWaitPolls = 100000; // x kSuspendHintNs = 2 s

// What the other roles need to know of a unit; posted by the weight producer.
struct UDesc {
  int32_t unit;                                // index in the unit list, -1 = no more work
  int32_t row_tile, tok0, ntok, g0, ng, split;
  uint32_t bits;                               // bitwidth of matrix 0 | bitwidth of matrix 1 << 8
};
static_assert(sizeof(UDesc) == 32, "UDesc layout");

struct Ctrl {                                  // lives at the start of dynamic shared memory
  // One full barrier per ring slot (armed by the weight producer).  A slot is handed back by sixteen arrivals:
  // four per tile of the chunk, from the warps of the dequantizer group that read the tile, or from the MMA
  // issuer that read a 16-bit tile (one tcgen05.commit plus three plain arrivals); for a chunk of fewer than
  // four tiles the producer itself makes up the difference when it arms the slot.
  unsigned long long full[kMaxSlots], empty[kMaxSlots];
  unsigned long long b_full[kMaxBSlots], b_empty[kMaxBSlots];
  unsigned long long a_full[kMaxASlots], a_empty[kMaxASlots];
  unsigned long long d_full[2], d_empty[2];     // two accumulator buffers (a wide token tile takes both)
  uint32_t tmem_base;
  volatile int abort_flag;
  volatile uint32_t issued;                    // chunks armed so far
  volatile uint32_t b_issued;                  // token tiles armed so far
  // Work list of this CTA: the weight producer claims units from a global counter and posts them here;
  // entry i & 31 is valid once sched_n > i (the producer is never more than a ring of slots ahead of the others).
  volatile uint32_t sched_n;
  // Set once the kernel ahead of this one in the stream has completed.  Until then a wait that runs out is not a
  // fault (the CTA may have been placed long before its inputs exist) and simply starts over.
  volatile uint32_t dep_ready;
  uint32_t pad_[2];
  UDesc sched[kSched];
};
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");

struct TmapSet {                               // token-tile copies: one map per tile height 16, 32, .. 128
  CUtensorMap m[8];
};

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_s(uint32_t bar_s) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_s) : "memory");
}
// one arrival by the threads for which `pred` holds (no branch around it)
__device__ __forceinline__ void mbar_arrive_if_s(uint32_t bar_s, bool pred) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %1, 0;\n\t"
      "@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar_s),
      "r"((uint32_t)pred)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_n_s(uint32_t bar_s, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx_s(uint32_t bar_s, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_s), "r"(bytes) : "memory");
}
// One bounded wait: up to `polls` try_waits, each of which sleeps inside the barrier unit for up to
// kSuspendHintNs (an arrival that does not complete the phase still wakes it, hence the loop).  The loop is
// inline PTX on purpose: an out-of-line slow path in a hot loop makes the compiler keep the loop's state in
// call-preserved registers.
__device__ __forceinline__ bool mbar_poll(uint32_t bar_s, uint32_t parity, uint32_t polls) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .u32 n;\n\t"
      "mov.u32 n, 0;\n"
      "PW_WAITN:\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "@p bra PW_DONEN;\n\t"
      "add.u32 n, n, 1;\n\t"
      "setp.lt.u32 q, n, %4;\n\t"
      "@q bra PW_WAITN;\n"
      "PW_DONEN:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar_s), "r"(parity), "r"(kSuspendHintNs), "r"(polls)
      : "memory");
  return ok != 0;
}
// Sleep-and-look until the shared-memory word at `addr_s` exceeds `value`: at least 64 ns per look, `looks` looks.
__device__ __forceinline__ bool flag_poll(uint32_t addr_s, uint32_t value, uint32_t looks) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t.reg .u32 v, k;\n\t"
      "mov.u32 k, 0;\n"
      "PW_FL:\n\t"
      "ld.volatile.shared.u32 v, [%1];\n\t"
      "setp.gt.u32 p, v, %2;\n\t"
      "@p bra PW_FLD;\n\t"
      "nanosleep.u32 64;\n\t"
      "add.u32 k, k, 1;\n\t"
      "setp.lt.u32 q, k, %3;\n\t"
      "@q bra PW_FL;\n"
      "PW_FLD:\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(addr_s), "r"(value), "r"(looks)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_g2s_s(uint32_t dst_s, const void* src, uint32_t bytes, uint32_t bar_s) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_s),
               "l"(src), "r"(bytes), "r"(bar_s)
               : "memory");
}
__device__ __forceinline__ void tma_2d_g2s_s(uint32_t dst_s, const CUtensorMap* map, int x, int y, uint32_t bar_s) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          dst_s),
      "l"(map), "r"(x), "r"(y), "r"(bar_s)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit_s(uint32_t bar_s) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_s) : "memory");
}
// Four consecutive k-steps issued from one asm block (the issuing thread gets few issue slots, so every
// instruction around an MMA counts).  Descriptors are passed as (lo, hi) words; only lo moves.
// TS: A in tensor memory at a_tmem (+a_step per k-step).  `acc0`: accumulate flag of the first k-step.
__device__ __forceinline__ void tc_mma_ts_burst4(uint32_t d_tmem, uint32_t a_tmem, uint32_t a_step, uint32_t b_lo,
                                                 uint32_t b_hi, uint32_t b_step, uint32_t idesc, uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p, t;\n\t.reg .b64 bd;\n\t.reg .b32 lo, a;\n\t"
      "setp.ne.b32 p, %7, 0;\n\t"
      "setp.eq.b32 t, 0, 0;\n\t"
      "mov.b64 bd, {%3, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %6, p;\n\t"
      "add.u32 lo, %3, %5;\n\tadd.u32 a, %1, %2;\n\tmov.b64 bd, {lo, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
      "add.u32 lo, lo, %5;\n\tadd.u32 a, a, %2;\n\tmov.b64 bd, {lo, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
      "add.u32 lo, lo, %5;\n\tadd.u32 a, a, %2;\n\tmov.b64 bd, {lo, %4};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(acc0)
      : "memory");
}
// SS: A in shared memory, descriptor (a_lo, a_hi), +a_step per k-step.
__device__ __forceinline__ void tc_mma_ss_burst4(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t a_step,
                                                 uint32_t b_lo, uint32_t b_hi, uint32_t b_step, uint32_t idesc,
                                                 uint32_t acc0) {
  asm volatile(
      "{\n\t.reg .pred p, t;\n\t.reg .b64 ad, bd;\n\t.reg .b32 la, lb;\n\t"
      "setp.ne.b32 p, %8, 0;\n\t"
      "setp.eq.b32 t, 0, 0;\n\t"
      "mov.b64 ad, {%1, %2};\n\tmov.b64 bd, {%4, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, p;\n\t"
      "add.u32 la, %1, %3;\n\tadd.u32 lb, %4, %6;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
      "add.u32 la, la, %3;\n\tadd.u32 lb, lb, %6;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
      "add.u32 la, la, %3;\n\tadd.u32 lb, lb, %6;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(acc0)
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
      "[%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// ---- the pieces every role shares -------------------------------------------------------------------
// A wait ran out: not a fault while the kernel ahead is still running, otherwise the CTA gives up.
__device__ __forceinline__ bool wait_failed(Ctrl* c, int32_t* status) {
  if (!c->dep_ready) return false;               // start over
  c->abort_flag = 1;
  atomicMax(status, (int)PW_ERR_TIMEOUT);
  return true;
}
__device__ __forceinline__ bool wait_bar(uint32_t bar_s, uint32_t parity, uint32_t polls, Ctrl* c, int32_t* status) {
  while (!mbar_poll(bar_s, parity, polls))
    if (wait_failed(c, status)) return false;
  return true;
}
__device__ __forceinline__ bool wait_flag(const volatile uint32_t* flag, uint32_t value, uint32_t polls, Ctrl* c,
                                          int32_t* status) {
  if (*flag > value) return true;
  const uint32_t looks = polls < (1u << 24) ? polls << 8 : 0xffffffffu;
  while (!flag_poll(smem_u32(const_cast<uint32_t*>(flag)), value, looks))
    if (wait_failed(c, status)) return false;
  return true;
}
// Entry i of this CTA's work list (bounded wait until the weight producer has posted it).
__device__ __forceinline__ bool get_desc(uint32_t i, uint32_t polls, Ctrl* c, int32_t* status, UDesc& d) {
  if (!wait_flag(&c->sched_n, i, polls, c, status)) return false;
  const uint4* p = reinterpret_cast<const uint4*>(&c->sched[i & (kSched - 1)]);
  const uint4 a = p[0], b = p[1];
  d.unit = (int32_t)a.x;
  d.row_tile = (int32_t)a.y;
  d.tok0 = (int32_t)a.z;
  d.ntok = (int32_t)a.w;
  d.g0 = (int32_t)b.x;
  d.ng = (int32_t)b.y;
  d.split = (int32_t)b.z;
  d.bits = b.w;
  return true;
}

// Chunks: tiles per chunk = 1 << chunk_log(bits).
// (a bit-plane tile, flagged by kPlanesFlag in the unit's bitwidth byte, is gathered from up to four places and travels alone)
constexpr uint32_t kPlanesFlag = 0x40;
__device__ __forceinline__ uint32_t chunk_log(uint32_t bits) { return (bits == 16 || (bits & kPlanesFlag)) ? 0u : bits == 8 ? 1u : 2u; }
// Chunk number inside a unit.  The producer walks the unit's groups in order and, at every group that starts a
// chunk of a matrix, issues that chunk (matrix 0 first): chunk i of matrix 0 is preceded by its own earlier
// chunks and by the chunks of matrix 1 that start before its first group, and the other way round.
template <int NMAT>
__device__ __forceinline__ uint32_t chunk_seq(uint32_t m, uint32_t i, uint32_t l0, uint32_t l1) {
  if (NMAT == 1) return i;
  if (m == 0) return i + (((i << l0) + (1u << l1) - 1u) >> l1);
  return i + ((i << l1) >> l0) + 1u;
}
// Position of a chunk in the ring, advanced incrementally.
struct Cursor {
  uint32_t seq, s, par;
};
__device__ __forceinline__ void cursor_to(Cursor& cu, uint32_t seq, uint32_t n_slots) {
  cu.s += seq - cu.seq;
  cu.seq = seq;
  while (cu.s >= n_slots) {
    cu.s -= n_slots;
    cu.par ^= 1u;
  }
}

// Shared-memory matrix descriptor, K-major, no swizzle.  A core matrix is 8 rows x 16 bytes (8 fp16
// along K) stored as 128 contiguous bytes; 8-row groups are 128 bytes apart (stride byte offset),
// the two K-halves of one MMA are `lbo_bytes` apart (leading byte offset).
__device__ __forceinline__ uint64_t make_kmajor_desc(uint32_t saddr, uint32_t lbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((128u >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version of sm_100
  return d;
}

struct KArgs {
  const DevRow* rows;                            // page-table rows of the layer (final before the call's first kernel)
  const Unit* units;
  const int32_t* n_units_ptr;
  int Rpad, nt_tile, n_bslots, n_slots;
  __half* ht;
  float* y;
  int H;
  size_t y_split_stride;
  int32_t* work_counter;
  int32_t* status;
  uint32_t wait_polls;                           // limit of every wait, in polls of kSuspendHintNs
  uint32_t hook;                                 // test hook: bit 0 = the token-tile producer stops before its second tile
};

// ---- dequantizers: the tiles of one unit that belong to one group -------------------------------------------
// Tile j of the unit sits in chunk j >> L of its matrix; a warp looks at a chunk's barrier once, decodes its
// tiles of the chunk and makes one arrival on the slot per tile.
template <int BITS, int NMAT, bool PLANES>
__device__ __forceinline__ bool dq_unit(Ctrl* c, const KArgs& ka, char* wring, uint32_t m, uint32_t j0, uint32_t stride,
                                        uint32_t ng, uint32_t seq_unit, uint32_t l0, uint32_t l1, Cursor& cu,
                                        uint32_t& uses, int r, int lane, uint32_t lane_addr, uint32_t af_s, uint32_t ae_s) {
  constexpr uint32_t L = PLANES ? 0u : BITS == 8 ? 1u : 2u;
  constexpr uint32_t TB = BITS * 2048 + 512;
  constexpr uint32_t META = PLANES ? (uint32_t)kPlaneSlotLut : BITS * 2048u;   // scales, then zero-points, of the tile's rows
  const uint32_t full_s = smem_u32(&c->full[0]), empty_s = smem_u32(&c->empty[0]);
  uint32_t cur = 0xffffffffu;
  const char* chunk = nullptr;
  uint32_t slot_empty_s = 0;
#pragma unroll 1
  for (uint32_t j = j0; j < ng; j += stride) {
    const uint32_t ci = j >> L;
    if (ci != cur) {
      cur = ci;
      const uint32_t seq = seq_unit + chunk_seq<NMAT>(m, ci, l0, l1);
      cursor_to(cu, seq, (uint32_t)ka.n_slots);
      // a chunk's barrier is looked at only once the producer is known to have armed it: the phase parity
      // cannot tell an old phase of the slot from the chunk's own
      if (!wait_flag(&c->issued, seq, ka.wait_polls, c, ka.status)) return false;
      if (!wait_bar(full_s + 8 * cu.s, cu.par, ka.wait_polls, c, ka.status)) return false;
      chunk = wring + cu.s * kSlotBytes;
      slot_empty_s = empty_s + 8 * cu.s;
    }
    const char* tile = chunk + (j & ((1u << L) - 1u)) * TB;
    const uint4* row_units = reinterpret_cast<const uint4*>(tile) + r;
    const __half2 s2 = __half2half2(*reinterpret_cast<const __half*>(tile + META + 2 * r));
    const __half2 z2 = __half2half2(*reinterpret_cast<const __half*>(tile + META + 256 + 2 * r));
    __half2 w[32];
    if constexpr (PLANES) decode_half_planes<BITS>(tile, r, 0, s2, z2, w);
    else decode_half<BITS>(row_units, 0, s2, z2, w);
    // The operand slot is free once the MMAs of the group's previous tile have read it; they ran while the
    // half above was being decoded.
    if (!wait_bar(ae_s, (uses & 1u) ^ 1u, ka.wait_polls, c, ka.status)) return false;
    ++uses;
    tc_fence_after();
    tmem_st32(lane_addr, w);
    if constexpr (PLANES) decode_half_planes<BITS>(tile, r, 1, s2, z2, w);
    else decode_half<BITS>(row_units, 1, s2, z2, w);
    __syncwarp();
    mbar_arrive_if_s(slot_empty_s, lane == 0);     // this warp has read its rows of the tile
    tmem_st32(lane_addr + 32, w);
    // hand the tile over: both stores have landed, then one arrival per warp
    tmem_wait_st();
    tc_fence_before();
    __syncwarp();
    mbar_arrive_if_s(af_s, lane == 0);
  }
  return true;
}

// ---- epilogue of token columns [c_begin, c_end) of one unit, one accumulator row per thread ------------------
template <int PHASE>
__device__ __forceinline__ void epilogue_cols(const KArgs& ka, const UDesc& d, uint32_t dbase, int npart, uint32_t written,
                                              int nb_rows, int row, int c_begin, int c_end) {
  for (int c0 = c_begin; c0 < c_end; c0 += 16) {
    float a[16], b[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) a[j] = b[j] = 0.0f;
    for (int p = 0; p < npart; ++p) {              // add the issuers' partial sums, in order
      if (!((written >> p) & 1u)) continue;
      float t[16];
      tmem_ld16(dbase + p * nb_rows + c0, t);
      tmem_wait_ld();
#pragma unroll
      for (int j = 0; j < 16; ++j) a[j] = __fadd_rn(a[j], t[j]);
      if (PHASE == 0) {
        tmem_ld16(dbase + (npart + p) * nb_rows + c0, t);
        tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 16; ++j) b[j] = __fadd_rn(b[j], t[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      const int nn = c0 + j;
      if (nn < d.ntok) {
        if (PHASE == 0) {
          // SwiGLU: silu(gate) * up; the result is rounded to fp16, so the fast exponential and
          // division (relative error ~1e-6) change nothing that survives the rounding
          const float hval = __fmul_rn(__fdividef(a[j], __fadd_rn(1.0f, __expf(-a[j]))), b[j]);
          ka.ht[((size_t)(row >> 3) * ka.Rpad + d.tok0 + nn) * 8 + (row & 7)] = __float2half_rn(hval);
        } else {
          ka.y[(size_t)d.split * ka.y_split_stride + (size_t)(d.tok0 + nn) * ka.H + row] = a[j];
        }
      }
    }
  }
}

// PHASE 0: units of (expert, 128 FFN rows, token tile): gate and up pages -> Ht.
// PHASE 1: units of (expert, 128 hidden rows, token tile, K range): down page -> Y[split].
// PLANES: the instantiation that also reads overlaid bit-plane blocks; launched only for a layer that has one (the
// extra code paths cost the ordinary ones instruction-cache room).
template <int PHASE, bool HELP, bool PLANES>
__global__ void __launch_bounds__(kThreads, 1) ffn_tc_kernel(const __grid_constant__ KArgs ka, const __grid_constant__ TmapSet tmaps) {
  extern __shared__ __align__(1024) char smem[];
  Ctrl* c = reinterpret_cast<Ctrl*>(smem);
  char* wring = smem + kCtrlBytes;
  const int n_slots = ka.n_slots, n_bslots = ka.n_bslots, nt_tile = ka.nt_tile;
  char* bslots = wring + n_slots * kSlotBytes;
  const int bslot_bytes = nt_tile * 256;
  constexpr int NMAT = PHASE == 0 ? 2 : 1;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int32_t* status = ka.status;
  const uint32_t polls = ka.wait_polls;
  // tensor-memory columns: partial accumulators first ([matrix][partial][nt_tile]), dequantized-operand
  // slots after them.  Partials per matrix: as many as issuers per matrix, while the operand slots still fit.
  constexpr int IPM = kIssuers / NMAT;           // issuers per matrix = dequantizer groups per matrix
  int npart = IPM;
  while (npart > 1 && NMAT * npart * nt_tile + kMaxASlots * 64 > kTmemCols) npart >>= 1;
  const int n_issuers = NMAT * npart;            // active issuers
  const int acol = NMAT * npart * nt_tile;       // the operand slot of group g sits at acol + 64 * g

  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxSlots; ++i) {
      mbar_init(&c->full[i], 1);
      mbar_init(&c->empty[i], kChunkArrivals);
    }
    for (int i = 0; i < kMaxBSlots; ++i) {
      mbar_init(&c->b_full[i], 1);
      mbar_init(&c->b_empty[i], NMAT);             // one issuer per matrix multiplies a token tile
    }
    for (int i = 0; i < kMaxASlots; ++i) {
      mbar_init(&c->a_full[i], 4);                // the four warps of the group that owns the slot
      mbar_init(&c->a_empty[i], 1);                // the issuer that serves the group
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&c->d_full[i], n_issuers);
      mbar_init(&c->d_empty[i], HELP ? 8 : 4);    // epilogue warps (+ the issuer warps when they share the epilogue)
    }
    c->abort_flag = 0;
    c->issued = 0;
    c->b_issued = 0;
    c->sched_n = 0;
    c->dep_ready = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&c->tmem_base)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = c->tmem_base;
  // This CTA may have been placed while the kernel before this one is still finishing on other SMs.  Work
  // counters, page-table rows and the unit counts were written two or more kernels back and are final (see
  // grid_dep_sync).  What the kernel directly ahead writes is not: the token rows (both kernels; the
  // token-tile producer waits for them) and the gate/up unit list (PHASE 0; the weight producer waits).
  // Nothing else reads global memory that a kernel of this call writes: the other roles learn of their units
  // from the weight producer, through shared memory.

  if (warp == kWarpW) {
    // ---------------- weight producer ----------------
    if (lane == 0) {
      if (PHASE == 0) {
        grid_dep_sync();
        c->dep_ready = 1;
      }
      const int n_units = ka.n_units_ptr[PHASE];
      const int G = gridDim.x;
      const uint32_t wring_s = smem_u32(wring), full_s = smem_u32(&c->full[0]), empty_s = smem_u32(&c->empty[0]);
      uint32_t seq = 0, s = 0, pass = 0;           // number and slot of the next chunk, laps around the ring
      int u = (int)blockIdx.x < n_units ? (int)blockIdx.x : -1;   // unit blockIdx.x first, then whatever the counter hands out
      bool ok = true;
      for (uint32_t i = 0; ok; ++i) {
        UDesc d;
        d.unit = u;
        d.row_tile = d.tok0 = d.ntok = d.g0 = d.ng = d.split = 0;
        d.bits = 0;
        const char* src[NMAT];
        const char* pb1[NMAT];                      // bit-plane blocks: the BIT1 and BIT0 buffers
        const char* pb0[NMAT];
        uint32_t tb[NMAT], lg[NMAT], pq[NMAT];      // pq: bitwidth a bit-plane block is read at, 0 = an ordinary page
        if (u >= 0) {
          // (the unit list may have been written by the kernel directly ahead: read around the non-coherent path)
          const int4* up = reinterpret_cast<const int4*>(ka.units + u);
          const int4 u0 = __ldcg(up), u1 = __ldcg(up + 1);
          d.row_tile = u0.y;
          d.tok0 = u0.z;
          d.ntok = u0.w;
          d.g0 = u1.x;
          d.ng = u1.y - u1.x;
          d.split = u1.z;
#pragma unroll
          for (int m = 0; m < NMAT; ++m) {
            const DevRow row = ka.rows[u0.x * 3 + (PHASE == 0 ? m : 2)];
            const bool planes = PLANES && row.valid == 2;
            const uint32_t ubits = row.bits | (planes ? kPlanesFlag : 0u);
            d.bits |= ubits << (8 * m);
            pq[m] = planes ? row.bits : 0u;
            tb[m] = planes ? (uint32_t)kPlaneTopTile : (uint32_t)tile_bytes((int)row.bits);
            lg[m] = chunk_log(ubits);
            // consecutive groups of a row tile are consecutive tiles of the page
            const size_t tile = (size_t)d.row_tile * (row.cols / kGroup) + d.g0;
            src[m] = reinterpret_cast<const char*>(row.codes) + tile * tb[m];
            pb1[m] = reinterpret_cast<const char*>(row.bit1) + tile * kPlaneBitTile;
            pb0[m] = reinterpret_cast<const char*>(row.bit0) + tile * kPlaneBitTile;
          }
        }
        UDesc* slot = &c->sched[i & (kSched - 1)];
        *slot = d;
        __threadfence_block();
        c->sched_n = i + 1;
        if (u < 0) break;
        const uint32_t ng = (uint32_t)d.ng;
        const uint32_t claim_at = ng >> 1;
        int claimed = 0;
#pragma unroll 1
        for (uint32_t g = 0; ok && g < ng; ++g) {
          // claim the next unit half-way through this one: the answer is back long before it is needed
          if (g == claim_at) claimed = atomicAdd(ka.work_counter, 1) + G;
#pragma unroll
          for (int m = 0; m < NMAT; ++m) {
            if (g & ((1u << lg[m]) - 1u)) continue;
            const uint32_t left = ng - g, full_n = 1u << lg[m];
            const uint32_t nt = left < full_n ? left : full_n;
            const uint32_t q = PLANES ? pq[m] : 0u;
            const uint32_t bytes = q ? (uint32_t)kPlaneTopCodes + 512u + (q - 2u) * (uint32_t)kPlaneBitTile : nt * tb[m];
            const uint32_t es = empty_s + 8 * s, fs = full_s + 8 * s;
            if (pass) ok = wait_bar(es, (pass - 1) & 1, polls, c, status);
            if (!ok) break;
            if (nt < 4) mbar_arrive_n_s(es, (4 - nt) * 4);   // a short chunk: the arrivals its missing tiles would make
            mbar_expect_tx_s(fs, bytes);
            const uint32_t slot_s = wring_s + s * kSlotBytes;
            if (q) {
              // a bit-plane tile read at q bits: the top codes, the planes below them that q needs, and the
              // lookup-table state of q -- only the first q bits of every weight leave HBM
              bulk_g2s_s(slot_s, src[m], kPlaneTopCodes, fs);
              bulk_g2s_s(slot_s + kPlaneSlotLut, src[m] + plane_lut_offset((int)q), 512, fs);
              if (q >= 3) bulk_g2s_s(slot_s + kPlaneSlotBit1, pb1[m], kPlaneBitTile, fs);
              if (q == 4) bulk_g2s_s(slot_s + kPlaneSlotBit0, pb0[m], kPlaneBitTile, fs);
              src[m] += kPlaneTopTile;
              pb1[m] += kPlaneBitTile;
              pb0[m] += kPlaneBitTile;
            } else {
              bulk_g2s_s(slot_s, src[m], bytes, fs);
              src[m] += bytes;
            }
            c->issued = ++seq;
            if (++s == (uint32_t)n_slots) {
              s = 0;
              ++pass;
            }
          }
        }
        u = claimed < n_units ? claimed : -1;
      }
    }
  } else if (warp == kWarpB) {
    // ---------------- token-tile producer ----------------
    if (lane == 0) {
      grid_dep_sync();
      grid_dep_trigger();
      if (PHASE == 1) c->dep_ready = 1;
      const uint32_t bslots_s = smem_u32(bslots), bf_s = smem_u32(&c->b_full[0]), be_s = smem_u32(&c->b_empty[0]);
      uint32_t bcount = 0, bs = 0, bpass = 0;
      bool ok = true;
      for (uint32_t i = 0; ok; ++i) {
        UDesc d;
        if (!get_desc(i, polls, c, status, d) || d.unit < 0) break;
        const int nb_rows = (d.ntok + 15) & ~15;
        const CUtensorMap* map = &tmaps.m[(nb_rows >> 4) - 1];
#pragma unroll 1
        for (int g = d.g0; ok && g < d.g0 + d.ng; ++g) {
          if ((ka.hook & 1u) && bcount == 1) {     // test hook: leave the tile unarmed, so that the waits on it run out
            ok = false;
            break;
          }
          // token tile of this group: 16 K-chunks x nb_rows rows x 16 bytes, one 2-D copy
          if (bpass) ok = wait_bar(be_s + 8 * bs, (bpass - 1) & 1, polls, c, status);
          if (!ok) break;
          mbar_expect_tx_s(bf_s + 8 * bs, nb_rows * 256);
          tma_2d_g2s_s(bslots_s + bs * (uint32_t)bslot_bytes, map, d.tok0 * 2, g * 16, bf_s + 8 * bs);
          c->b_issued = ++bcount;
          if (++bs == (uint32_t)n_bslots) {
            bs = 0;
            ++bpass;
          }
        }
      }
    }
  } else if (warp >= kWarpMma && warp < kWarpMma + kIssuers) {
    // ---------------- MMA issuers ----------------
    // Tile k of a matrix (counted over all units) belongs to issuer k mod npart of that matrix, which issues
    // all eight k-steps of it into its own partial accumulator; a quantized tile k is dequantized by the
    // matrix's group k mod IPM, so with npart == IPM every dequantizer group has an issuer of its own.
    // The epilogue adds the partials.  With HELP every lane follows the units (the warp shares the epilogue of
    // wide units, taking the upper half of the token columns of its lane quarter); lane 0 issues.
    const int iss = warp - kWarpMma;
    const int my_m = iss / IPM, my_j = iss % IPM;
    const bool issuing = my_j < npart;
    if ((HELP || (lane == 0 && issuing))) {
      const int hq = warp & 3;
      const uint32_t hlane_addr = tmem + ((uint32_t)(hq * 32) << 16);
      uint32_t seq_unit = 0;                        // chunks before the current unit
      uint32_t base = 0;                            // tiles of one matrix (= token tiles) before the current unit
      uint32_t upar = 0;                            // per group: parity of the next use of its operand slot
      // Accumulators: partial (m, j) of a unit sits at buffer base + (m * npart + j) * nb_rows.  A unit whose
      // accumulators fit half of the accumulator columns takes one of two buffers in turn, so that its MMAs
      // overlap the epilogue of the unit before it; a wider unit takes both.
      uint32_t dtoggle = 0, duse0 = 0, duse1 = 0;
      const uint32_t desc_hi = (uint32_t)(make_kmajor_desc(0, 0) >> 32);
      const uint32_t b_lo_base = smem_u32(bslots) >> 4;
      const uint32_t w_lo_base = smem_u32(wring) >> 4;
      const uint32_t af_s = smem_u32(&c->a_full[0]), ae_s = smem_u32(&c->a_empty[0]);
      const uint32_t bf_s = smem_u32(&c->b_full[0]), be_s = smem_u32(&c->b_empty[0]);
      const uint32_t full_s = smem_u32(&c->full[0]), empty_s = smem_u32(&c->empty[0]);
      const uint32_t df_s = smem_u32(&c->d_full[0]), de_s = smem_u32(&c->d_empty[0]);
      const uint32_t a_base = tmem + acol;
      Cursor cu = {0, 0, 0};
      Cursor bp = {0, 0, 0};
      bool ok = true;
      for (uint32_t i = 0; ok; ++i) {
        UDesc d;
        if (!get_desc(i, polls, c, status, d) || d.unit < 0) break;
        const uint32_t bits0 = d.bits & 0xffu, bits1 = NMAT == 2 ? (d.bits >> 8) & 0xffu : bits0;
        const uint32_t my_bits = my_m ? bits1 : bits0;
        const uint32_t l0 = chunk_log(bits0), l1 = chunk_log(bits1);
        const uint32_t ng = (uint32_t)d.ng;
        const uint32_t nch = ((ng + (1u << l0) - 1u) >> l0) + (NMAT == 2 ? ((ng + (1u << l1) - 1u) >> l1) : 0u);
        const int nb_rows = (d.ntok + 15) & ~15;
        const bool wide = NMAT * npart * nb_rows > acol / 2;
        const uint32_t dbuf = wide ? 0u : dtoggle;
        if (!wide) dtoggle ^= 1u;
        if (lane == 0 && issuing) {
          const uint32_t idesc = (1u << 4) | ((uint32_t)(nb_rows >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
          // B descriptor: leading byte offset = nb_rows * 16 (field at bit 16), advance 2 * nb_rows k-chunk units per k-step
          const uint32_t b_lo_unit = b_lo_base | ((uint32_t)nb_rows << 16);
          const uint32_t b_step = (uint32_t)(2 * nb_rows);
          const uint32_t a_lo_lbo = (2048u >> 4) << 16;                 // A descriptor (16-bit tiles): LBO 2048 B
          const uint32_t d_t = tmem + dbuf * (uint32_t)(acol / 2) + (uint32_t)((my_m * npart + my_j) * nb_rows);
          // the epilogue has drained the buffer(s) this unit accumulates into
          if (wide || dbuf == 0) ok = wait_bar(de_s, (duse0 & 1) ^ 1, polls, c, status);
          if (ok && (wide || dbuf == 1)) ok = wait_bar(de_s + 8, (duse1 & 1) ^ 1, polls, c, status);
          if (ok) {
            tc_fence_after();
            uint32_t later = 0;                          // becomes 1 after my first tile: accumulate onto earlier ones
            // my first tile of the unit, then every npart-th
#pragma unroll 1
            for (uint32_t j = ((uint32_t)my_j - base) & (uint32_t)(npart - 1); j < ng; j += (uint32_t)npart) {
              // the token tile of this group (a tile is looked at only once it is known to have been armed)
              const uint32_t bt = base + j;
              cursor_to(bp, bt, (uint32_t)n_bslots);
              ok = wait_flag(&c->b_issued, bt, polls, c, status) && wait_bar(bf_s + 8 * bp.s, bp.par, polls, c, status);
              if (!ok) break;
              const uint32_t b_lo = b_lo_unit + bp.s * (uint32_t)(bslot_bytes >> 4);
              if (my_bits == 16) {
                // the whole tile lies in one slot as a K-major core-matrix image (k-steps 4 KB apart)
                const uint32_t seq = seq_unit + chunk_seq<NMAT>((uint32_t)my_m, j, l0, l1);
                cursor_to(cu, seq, (uint32_t)n_slots);
                ok = wait_flag(&c->issued, seq, polls, c, status) && wait_bar(full_s + 8 * cu.s, cu.par, polls, c, status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_lo = (w_lo_base + cu.s * (kSlotBytes >> 4)) | a_lo_lbo;
                tc_mma_ss_burst4(d_t, a_lo, desc_hi, 256, b_lo, desc_hi, b_step, idesc, later);
                tc_mma_ss_burst4(d_t, a_lo + 4 * 256, desc_hi, 256, b_lo + 4 * b_step, desc_hi, b_step, idesc, 1u);
                mbar_arrive_n_s(empty_s + 8 * cu.s, 3);  // with the commit: the four arrivals of the tile
                tc_commit_s(empty_s + 8 * cu.s);
              } else {
                // the group that dequantizes this tile, and the parity of this use of its operand slot
                const uint32_t grp = NMAT == 2 ? 2u * (uint32_t)my_m + (bt & 1u) : (bt & 3u);
                const uint32_t use_par = (upar >> grp) & 1u;
                upar ^= 1u << grp;
                const uint32_t a_t = a_base + grp * 64;
                ok = wait_bar(af_s + 8 * grp, use_par, polls, c, status);
                if (!ok) break;
                tc_fence_after();
                // all eight k-steps of the tile, then one commit hands the group's operand slot back
                tc_mma_ts_burst4(d_t, a_t, 8, b_lo, desc_hi, b_step, idesc, later);
                tc_mma_ts_burst4(d_t, a_t + 32, 8, b_lo + 4 * b_step, desc_hi, b_step, idesc, 1u);
                tc_commit_s(ae_s + 8 * grp);
              }
              tc_commit_s(be_s + 8 * bp.s);
              later = 1;
            }
          }
          if (ok) {
            if (wide || dbuf == 0) tc_commit_s(df_s);
            if (wide || dbuf == 1) tc_commit_s(df_s + 8);
          }
        }
        const uint32_t par0 = duse0 & 1u, par1 = duse1 & 1u;     // phases of d_full this unit completes
        if (wide || dbuf == 0) ++duse0;
        if (wide || dbuf == 1) ++duse1;
        if (HELP) {
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
          // every issuer warp sees every phase of the accumulator barriers, also of the narrow units it has no
          // part in: it must not run ahead of the epilogue by more than the phase parity can tell apart
          if (wide || dbuf == 0) ok = wait_bar(df_s, par0, polls, c, status);
          if (ok && (wide || dbuf == 1)) ok = wait_bar(df_s + 8, par1, polls, c, status);
          if (!ok) break;
          if (wide) {
            tc_fence_after();
            uint32_t written = 0;
            for (int p = 0; p < npart; ++p)
              if ((((uint32_t)p - base) & (uint32_t)(npart - 1)) < ng) written |= 1u << p;
            const int half = ((nb_rows / 16 + 1) / 2) * 16;         // the epilogue warps take [0, half)
            epilogue_cols<PHASE>(ka, d, hlane_addr, npart, written, nb_rows, d.row_tile * kTileRows + hq * 32 + lane, half,
                                 nb_rows);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) {
              mbar_arrive_s(de_s);
              mbar_arrive_s(de_s + 8);
            }
          }
        }
        base += ng;
        seq_unit += nch;
      }
    }
  } else if (warp < kDqWarps) {
    // ---------------- dequantize ----------------
    // Four groups of four warps, each taking every other quantized tile of one matrix (every fourth when
    // the unit has a single matrix).  Warp q of a group owns rows (= TMEM lanes) 32q .. 32q+31 of the tile,
    // one row per thread.  Each group has one operand slot (64 columns: both K-halves of a tile): it stores the
    // two halves as it decodes them and hands the slot over once per tile; while the issuer's eight MMAs read
    // it, the group decodes the first half of its next tile in registers.
    const int grp = warp >> 2, q = warp & 3;
    const int r = q * 32 + lane;                     // weight row inside the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16) + acol + grp * 64;
    const uint32_t qm = NMAT == 2 ? (uint32_t)(grp >> 1) : 0u;         // the matrix this group serves
    const uint32_t gsub = NMAT == 2 ? (uint32_t)(grp & 1) : (uint32_t)grp;   // which of that matrix's groups
    constexpr uint32_t kStride = NMAT == 2 ? 2 : 4;  // groups per matrix = distance between my tiles
    const uint32_t af_s = smem_u32(&c->a_full[grp]), ae_s = smem_u32(&c->a_empty[grp]);
    uint32_t seq_unit = 0;                           // chunks before the current unit
    uint32_t base = 0;                               // tiles of one matrix before the current unit
    uint32_t uses = 0;                               // tiles I have taken so far (parity of my slot's use)
    Cursor cu = {0, 0, 0};
    bool ok = true;
    for (uint32_t i = 0; ok; ++i) {
      UDesc d;
      if (!get_desc(i, polls, c, status, d) || d.unit < 0) break;
      const uint32_t bits0 = d.bits & 0xffu, bits1 = NMAT == 2 ? (d.bits >> 8) & 0xffu : bits0;
      const uint32_t bits = qm ? bits1 : bits0;
      const uint32_t l0 = chunk_log(bits0), l1 = chunk_log(bits1);
      const uint32_t ng = (uint32_t)d.ng;
      const uint32_t nch = ((ng + (1u << l0) - 1u) >> l0) + (NMAT == 2 ? ((ng + (1u << l1) - 1u) >> l1) : 0u);
      // Tile k of a matrix (counted over all units) goes to that matrix's group k mod kStride: my first one
      // in this unit is tile j0, then every kStride-th.  (The MMA reads 16-bit tiles straight from shared memory.)
      const uint32_t j0 = (gsub - base) & (kStride - 1);
      switch (bits) {
        case 8: ok = dq_unit<8, NMAT, false>(c, ka, wring, qm, j0, kStride, ng, seq_unit, l0, l1, cu, uses, r, lane, lane_addr, af_s, ae_s); break;
        case 4: ok = dq_unit<4, NMAT, false>(c, ka, wring, qm, j0, kStride, ng, seq_unit, l0, l1, cu, uses, r, lane, lane_addr, af_s, ae_s); break;
        case 3: ok = dq_unit<3, NMAT, false>(c, ka, wring, qm, j0, kStride, ng, seq_unit, l0, l1, cu, uses, r, lane, lane_addr, af_s, ae_s); break;
        case 2: ok = dq_unit<2, NMAT, false>(c, ka, wring, qm, j0, kStride, ng, seq_unit, l0, l1, cu, uses, r, lane, lane_addr, af_s, ae_s); break;
#define PW_PLANE_CASE(Q) case kPlanesFlag | Q: if constexpr (PLANES) ok = dq_unit<Q, NMAT, true>(c, ka, wring, qm, j0, kStride, ng, seq_unit, l0, l1, cu, uses, r, lane, lane_addr, af_s, ae_s); break;
        PW_PLANE_CASE(4)
        PW_PLANE_CASE(3)
        PW_PLANE_CASE(2)
#undef PW_PLANE_CASE
        default: break;
      }
      base += ng;
      seq_unit += nch;
    }
  } else if (warp >= kWarpEpi) {
    // ---------------- epilogue ----------------
    const int q = warp & 3;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    const uint32_t df_s = smem_u32(&c->d_full[0]), de_s = smem_u32(&c->d_empty[0]);
    uint32_t base = 0;                               // tiles of one matrix before the current unit
    uint32_t dtoggle = 0, duse0 = 0, duse1 = 0;      // accumulator buffers: the issuers' rule, replayed
    bool ok = true;
    for (uint32_t i = 0; ok; ++i) {
      UDesc d;
      if (!get_desc(i, polls, c, status, d) || d.unit < 0) break;
      const int nb_rows = (d.ntok + 15) & ~15;
      const bool wide = NMAT * npart * nb_rows > acol / 2;
      const uint32_t dbuf = wide ? 0u : dtoggle;
      if (!wide) dtoggle ^= 1u;
      if (wide || dbuf == 0) ok = wait_bar(df_s, duse0 & 1, polls, c, status);
      if (ok && (wide || dbuf == 1)) ok = wait_bar(df_s + 8, duse1 & 1, polls, c, status);
      if (!ok) break;
      tc_fence_after();
      // partial accumulator p holds the tiles base + j with (base + j) mod npart == p: it has been written in
      // this unit only if there is such a j below the unit's group count
      const uint32_t ng = (uint32_t)d.ng;
      uint32_t written = 0;
      for (int p = 0; p < npart; ++p)
        if ((((uint32_t)p - base) & (uint32_t)(npart - 1)) < ng) written |= 1u << p;
      base += ng;
      // with helpers, the issuer warps take the upper half of the token columns of a wide unit
      const int c_end = HELP && wide ? ((nb_rows / 16 + 1) / 2) * 16 : nb_rows;
      epilogue_cols<PHASE>(ka, d, lane_addr + dbuf * (uint32_t)(acol / 2), npart, written, nb_rows,
                           d.row_tile * kTileRows + q * 32 + lane, 0, c_end);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        // (a narrow unit has no helpers: this warp arrives for the issuer warp of its lane quarter as well)
        const uint32_t n_arr = HELP && !wide ? 2u : 1u;
        if (wide || dbuf == 0) mbar_arrive_n_s(de_s, n_arr);
        if (wide || dbuf == 1) mbar_arrive_n_s(de_s + 8, n_arr);
      }
      if (wide || dbuf == 0) ++duse0;
      if (wide || dbuf == 1) ++duse1;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kWarpMma) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
  }
}

// ---- host side ---------------------------------------------------------------------------------
struct TcState {
  TmapSet xt, ht;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Maps over a k-chunk-major operand buffer [n_chunks][Rpad] of 16-byte units, seen as 8-byte
// elements: box = (2 * rows) x 16 chunks, so that one copy lands [16][rows][16 B] in shared memory.
static bool make_maps(EncodeTiledFn enc, void* base, int n_chunks, int Rpad, TmapSet* out) {
  for (int i = 0; i < 8; ++i) {
    const int rows = 16 * (i + 1);
    cuuint64_t gdim[2] = {(cuuint64_t)Rpad * 2, (cuuint64_t)n_chunks};
    cuuint64_t gstride[1] = {(cuuint64_t)Rpad * 16};
    cuuint32_t box[2] = {(cuuint32_t)rows * 2, 16};
    cuuint32_t estr[2] = {1, 1};
    if (enc(&out->m[i], CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, base, gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) !=
        CUDA_SUCCESS)
      return false;
  }
  return true;
}

typedef void (*FfnKernel)(const KArgs, const TmapSet);
static FfnKernel ffn_kernel_of(int phase, int help, int planes) {
  static const FfnKernel tab[8] = {ffn_tc_kernel<0, false, false>, ffn_tc_kernel<1, false, false>, ffn_tc_kernel<0, true, false>,
                                   ffn_tc_kernel<1, true, false>,  ffn_tc_kernel<0, false, true>,  ffn_tc_kernel<1, false, true>,
                                   ffn_tc_kernel<0, true, true>,   ffn_tc_kernel<1, true, true>};
  return tab[phase + 2 * help + 4 * planes];
}

static pw_status tc_setup(pw_ctx* ctx) {
  if (ctx->tc_state) return PW_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  PW_CUDA_OK(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return PW_ERR_CUDA;
  TcState* st = new (std::nothrow) TcState();
  if (!st) return PW_ERR_NOMEM;
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  if (!make_maps(reinterpret_cast<EncodeTiledFn>(fn), ctx->base + w.xt, c.hidden / 8, w.Rpad, &st->xt) ||
      !make_maps(reinterpret_cast<EncodeTiledFn>(fn), ctx->base + w.ht, c.ffn / 8, w.Rpad, &st->ht)) {
    delete st;
    return PW_ERR_CUDA;
  }
  for (int i = 0; i < 8; ++i)
    PW_CUDA_OK(cudaFuncSetAttribute(ffn_kernel_of(i & 1, (i >> 1) & 1, (i >> 2) & 1), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kMaxDynSmem));
  ctx->tc_state = st;
  return PW_OK;
}

void tc_teardown(pw_ctx* ctx) {
  delete reinterpret_cast<TcState*>(ctx->tc_state);
  ctx->tc_state = nullptr;
}

int tensor_token_tile(const pw_ctx* ctx, int T, int k) {
  // An expert never holds more than T tokens.  Tiles of 128 tokens leave tensor memory for one partial
  // accumulator per matrix only (one MMA issuer per matrix): right when experts hold hundreds of tokens and
  // the MMAs are wide, wrong when most experts hold a few dozen.  So: 128 only if the average routed expert
  // holds more than 64 tokens, otherwise at most 64 (a busier expert then takes several tiles).
  int nt = (T + 15) & ~15;
  const long long avg = ((long long)T * k) / (ctx->cfg.n_experts > 0 ? ctx->cfg.n_experts : 1);
  const int cap = avg > 64 ? 128 : 64;
  if (nt > cap) nt = cap;
  return nt;
}

pw_status launch_ffn_tensor(pw_ctx* ctx, int layer, int T, int k, int nt_tile, int ksplit, cudaStream_t s) {
  const pw_config& c = ctx->cfg;
  const WsMap& w = ctx->ws;
  char* b = ctx->base;
  pw_status pst = tc_setup(ctx);
  if (pst != PW_OK) return pst;
  const TcState* st = reinterpret_cast<const TcState*>(ctx->tc_state);
  const int bslot_bytes = nt_tile * 256;
  // Shared-memory plan per kernel.  The issuers of a matrix work on as many token tiles at once as there are
  // partial accumulators per matrix (the kernel's own rule, repeated here); one more slot keeps a tile on its
  // way.  The rest of the 227 KB goes to the weight ring.
  int n_bslots[2], n_slots[2], smem[2];
  for (int phase = 0; phase < 2; ++phase) {
    const int nmat = phase == 0 ? 2 : 1;
    int npart = kIssuers / nmat;
    while (npart > 1 && nmat * npart * nt_tile + kMaxASlots * 64 > kTmemCols) npart >>= 1;
    n_bslots[phase] = npart + 1 > kMaxBSlots ? kMaxBSlots : npart + 1;
    int ns = (kMaxDynSmem - kCtrlBytes - n_bslots[phase] * bslot_bytes) / kSlotBytes;
    if (ns > kMaxSlots) ns = kMaxSlots;
    if (ns < 3) return PW_ERR_NOMEM;
    n_slots[phase] = ns;
    smem[phase] = kCtrlBytes + ns * kSlotBytes + n_bslots[phase] * bslot_bytes;
  }
  const int R = T * k + c.n_shared * T;
  KArgs ka;
  ka.rows = reinterpret_cast<const DevRow*>(b + w.table) + (size_t)layer * w.S * 3;
  ka.n_units_ptr = reinterpret_cast<const int32_t*>(b + w.n_units);
  ka.Rpad = w.Rpad;
  ka.nt_tile = nt_tile;
  ka.H = c.hidden;
  ka.status = reinterpret_cast<int32_t*>(b + w.status);
  ka.wait_polls = ctx->wait_polls ? ctx->wait_polls : kDefaultWaitPolls;
  ka.hook = ctx->test_hook;
  int32_t* work_counter = reinterpret_cast<int32_t*>(b + w.counter);   // [0] gate/up, [1] down; zeroed by the permute kernel
  timing_mark(ctx, PW_K_FFN_GATE_UP, s);
  // token tiles of 128 leave no second accumulator buffer: the variant whose issuer warps share the epilogue
  const bool help = nt_tile > 64;
  bool planes = false;                           // does the layer hold a bit-plane block?
  for (int e = 0; e < w.S && !planes; ++e)
    for (int u = 0; u < 3; ++u) planes |= ctx->host_rows[row_index(ctx, layer, e, u)].page.layout == PW_LAYOUT_PLANES;
  ka.units = reinterpret_cast<const Unit*>(b + w.units_gu);
  ka.n_bslots = n_bslots[0];
  ka.n_slots = n_slots[0];
  ka.ht = reinterpret_cast<__half*>(b + w.ht);
  ka.y = nullptr;
  ka.y_split_stride = 0;
  ka.work_counter = work_counter;
  PW_CUDA_OK(launch_dependent(ffn_kernel_of(0, help, planes), dim3(ctx->num_sms), dim3(kThreads),
                              (size_t)smem[0], s, ka, st->xt));
  timing_mark(ctx, PW_K_FFN_DOWN, s);
  ka.units = reinterpret_cast<const Unit*>(b + w.units_dn);
  ka.n_bslots = n_bslots[1];
  ka.n_slots = n_slots[1];
  ka.ht = nullptr;
  ka.y = reinterpret_cast<float*>(b + w.y);
  ka.y_split_stride = (size_t)R * c.hidden;
  ka.work_counter = work_counter + 1;
  ka.hook = 0;
  PW_CUDA_OK(launch_dependent(ffn_kernel_of(1, help, planes), dim3(ctx->num_sms), dim3(kThreads),
                              (size_t)smem[1], s, ka, st->ht));
  ctx->launches += 2;
  PW_CUDA_OK(cudaGetLastError());
  (void)ksplit;
  return PW_OK;
}

}  // namespace pw
