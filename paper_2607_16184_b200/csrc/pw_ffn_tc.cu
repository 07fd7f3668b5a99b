// Tensor-core expert FFN for sm_100a.
//
//   D[128 weight rows, N tokens] += W[128, 16] * X[N, 16]^T      (tcgen05.mma, kind::f16, fp32 in TMEM)
//
// Weight pages stream HBM -> shared memory with bulk async copies into a ring of 17 KB slots.  A "slot item"
// is one tile image of a quantized page (128 rows x one group: codes, scales, zero-points, 4.5 .. 16.5 KB,
// one copy) or one K-half (16 KB) of a 16-bit tile; slot item number seq lives in slot seq mod n_slots, so
// every role finds its own items from their numbers alone.  A 16-bit half is already in the tensor core's
// K-major core-matrix layout: the MMA reads it from shared memory as the A operand without any thread
// touching it.  A quantized tile is unpacked and dequantized in registers (one weight row per thread) and
// written to tensor memory, which the MMA then reads as its A operand.  The token tile (B operand) comes
// from the k-chunk-major operand buffers with one 2-D TMA copy per group.
//
// One persistent CTA per SM, 27 warps.  The control roles have short dependent instruction chains: they share
// the schedulers with the arithmetic-heavy dequantizers, and every instruction of theirs waits its turn, so each
// of them does as little per item as possible.  Each runs as a whole, converged warp on the same values, lane 0
// being a predicate on the instructions with an effect (copies, MMAs, commits, arrivals): the MMA, the bulk copy
// and the barrier operations take their operands from uniform registers, which a single lane inside a divergent
// branch can only fill by moving every operand over for every instruction.
//   warps 0-15   dequantize: four groups of four warps; tile k of a matrix goes to that matrix's group
//                k mod (groups per matrix); warp w owns TMEM lanes 32*(w%4).., one weight row per thread;
//                a group has one operand slot of 64 columns in tensor memory (a whole tile, K 0..127) and hands
//                it to its issuer once per tile, while it decodes the first half of its next tile in registers;
//   warps 16,18  weight producers: producer P arms the slot items with number = P mod 2 (which sit in the
//                slots = P mod 2) and issues their copies, as far ahead as the ring allows; producer 0 also
//                claims the CTA's units from a global counter and posts them (the unit and the bitwidths of its
//                pages) on the CTA's work list in shared memory, the only place the other roles learn of them;
//   warp 17      token-tile producer (its own few slots, never holds back the weight stream);
//   warps 19-22  MMA issuers (warp 19 also allocates tensor memory).  Issuing a tcgen05.mma costs its warp tens of
//                cycles whatever its size, so the issuers work in parallel: issuer j of a
//                matrix issues all eight k-steps of the tiles k = j mod (issuers per matrix) into its own
//                partial accumulator -- with as many issuers as groups, each dequantizer group has an
//                issuer of its own -- and no two threads ever accumulate into the same columns at the same time
//                (the SHARE instantiations let the two issuers of an accumulator take turns on it where a
//                unit's token tile is wide, see unit_accumulators);
//   warps 23-26  epilogue: adds the partials; SwiGLU -> fp16 operand of the down projection (PHASE 0), or the
//                fp32 split-K partial of the down projection (PHASE 1).  Narrow token tiles alternate
//                between two accumulator buffers, so the next unit's MMAs overlap the epilogue.
//                Token tiles wider than 64 leave no second buffer: the HELP instantiation, launched for
//                those, has the four issuer warps share the epilogue of every wide unit.
//                Wide token tiles also leave the gate/up kernel one accumulator per matrix: there the two issuers
//                of a matrix take turns on it, tile by tile (a turn word in shared memory between tcgen05 fences
//                keeps the MMAs of an accumulator in tile order), so that one issuer's waits and hand-backs run
//                while the other issues.
// The two kernels of a call overlap: the down kernel's CTAs are placed on the SMs the gate/up kernel's CTAs leave,
// stream their weight pages at once, and start a unit when the gate/up units that write the SwiGLU rows of its K
// range have been counted in (a counter per token tile and K range, raised by the gate/up epilogue behind a
// fence, read with an acquire load by the down kernel's token-tile producer); the down list goes K range
// outermost so that the ranges finished first are multiplied first.
// Every wait is bounded; when one runs out the CTA records PW_ERR_TIMEOUT in the status word, stops issuing
// work, frees its tensor memory and returns.
// A block in the overlaid bit-plane format (Sec. 2.2, Sec. 3.1) is a slot item like any quantized tile: its
// producer copies the leading two planes, the lookup-table state of the bitwidth the page table names, and only
// as many further planes as that bitwidth reads.  Layers that hold such a block run the PLANES instantiation, so
// that the ordinary one keeps its decode switch and its registers.
#include <cuda.h>

#include <cstddef>

#include <new>

#include "pw_common.cuh"
#include "pw_layout.cuh"

namespace pw {

constexpr int kSlotBytes = 17408;               // one ring slot: an 8-bit item (16 KB codes + 512 B) fits
constexpr int kMaxSlots = 16;
constexpr int kMaxASlots = 4;                  // operand slots in tensor memory, one per group (64 columns = a 128 x 128 tile)
constexpr int kMaxBSlots = 5;
constexpr int kCtrlBytes = 1536;
constexpr int kMaxDynSmem = 232448;            // 227 KB
constexpr int kDqWarps = 16;
constexpr int kWarpCodes = 16, kWarpTokens = 17, kWarpCodes2 = 18, kWarpMma = 19, kIssuers = 4, kWarpEpi = 23;
constexpr int kThreads = 864;
constexpr int kTmemCols = 512;
constexpr uint32_t kSuspendHintNs = 20000;                   // a blocked barrier wait sleeps up to this long per poll
constexpr uint32_t kDefaultWaitPolls = 100000;               // x kSuspendHintNs = 2 s
constexpr uint32_t kTestWaitPolls = 200;                     // 4 ms: the limit of the instantiation that the failure-path test runs

struct Ctrl {                                  // lives at the start of dynamic shared memory
  // One full barrier per ring slot (armed by the weight producer).  A slot is handed back either by the
  // four warps of the dequantizer group that read it, or by the MMA issuer that read a 16-bit half from it
  // (one tcgen05.commit plus three plain arrivals, so that both kinds complete the same four-arrival phase
  // and the weight producers need not remember who holds a slot).
  unsigned long long full[kMaxSlots], empty[kMaxSlots];
  unsigned long long b_full[kMaxBSlots], b_empty[kMaxBSlots];
  unsigned long long a_full[kMaxASlots], a_empty[kMaxASlots];
  unsigned long long d_full[2], d_empty[2];     // two accumulator buffers (a wide token tile takes both)
  uint32_t tmem_base;
  volatile int abort_flag;
  // Slot items with an even number are armed by weight producer 0, odd ones by producer 1 (the number of
  // slots is even, so each producer also owns every other slot).  issued[p]: producer p has armed all of
  // its slot items below this number.
  volatile uint32_t issued[2];
  volatile uint32_t b_issued;                  // token tiles armed so far (same purpose, for the token-tile slots)
  // Accumulators that two issuers share (wide token tiles leave room for fewer accumulators than issuers): tiles
  // issued on accumulator a so far.  The issuer of the next tile waits for its turn, so the MMAs of an accumulator
  // enter the tensor pipe in tile order whoever issues them.
  volatile uint32_t turn[4];
  // Work list of this CTA: the weight producer claims units from a global counter and posts them here;
  // entry i & 31 is valid once sched_n > i (the producer is never more than a ring of slots ahead of the others), -1 ends the list.
  volatile uint32_t sched_n;
  volatile int32_t sched_unit[32];
  // the posted units themselves (entry i & 15), with the bitwidths of their pages packed into the spare word: what
  // every role needs to know about a unit, so that only the producers read the unit list and the page table
  alignas(16) Unit desc[16];                   // read and written 16 bytes at a time
};
static_assert(offsetof(Ctrl, desc) % 16 == 0, "descriptor alignment");
static_assert(sizeof(Ctrl) <= kCtrlBytes, "control block");


struct TmapSet {                               // token-tile copies: one map per tile height 16, 32, .. 128
  CUtensorMap m[8];
};

// ---- PTX wrappers ----------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(unsigned long long* b, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(unsigned long long* b, uint32_t n) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(b)), "r"(n) : "memory");
}
// Bounded wait.  Returns false when the limit ran out (and then raises the abort; the other roles of the CTA,
// starved by the one that gave up, run into their own limits within the same second or two, and since every
// role has then been idle for at least a second no copy of
// the CTA is still in flight when it leaves).  Each poll is a try_wait with a
// suspend-time hint, so a waiting thread sleeps inside the barrier unit instead of spending issue slots (an
// arrival that does not complete the phase still wakes it, hence the loop); 100000 polls of up to kSuspendHintNs
// each are the 2 s limit.  The loop is inline and written in PTX on purpose: with an out-of-line slow path the
// call made the compiler keep each role's loop state -- for the dequantizers a vector of 32 results between
// decode and store -- in call-preserved registers and copy it around, which cost 2 % of the decode step.
// (the barrier is given by its shared-memory address: the control loops keep those in registers)
// LIM: polls before the wait gives up.  It is an immediate, and the failure path is two stores, on purpose: the
// limit carried in a register, or a retry loop around the wait, cost the dequantizers 5 % of the decode step.
template <uint32_t LIM>
__device__ __forceinline__ bool mbar_wait_s(uint32_t bar_s, uint32_t parity, Ctrl* c, int32_t* status) {
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
      : "r"(bar_s), "r"(parity), "r"(kSuspendHintNs), "n"(LIM)
      : "memory");
  if (!ok) {
    c->abort_flag = 1;
    atomicMax(status, (int)PW_ERR_TIMEOUT);
  }
  return ok != 0;
}
// Sleep-and-look until the shared-memory word at `addr_s` exceeds `value`: at least 64 ns per look, 256 looks per
// poll of the barrier limit.
template <uint32_t LIM>
__device__ __forceinline__ bool flag_wait(uint32_t addr_s, uint32_t value, Ctrl* c, int32_t* status) {
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
      : "r"(addr_s), "r"(value), "n"(LIM * 256u)
      : "memory");
  if (!ok) {
    c->abort_flag = 1;
    atomicMax(status, (int)PW_ERR_TIMEOUT);
  }
  return ok != 0;
}
// predicated forms (the whole warp runs the producer's code, one lane acts)
__device__ __forceinline__ void mbar_expect_tx_if_s(uint32_t bar_s, uint32_t bytes, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t@q mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar_s),
      "r"(bytes), "r"(on)
      : "memory");
}
__device__ __forceinline__ void bulk_g2s_if_s(uint32_t dst_s, const void* src, uint32_t bytes, uint32_t bar_s, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %4, 0;\n\t"
      "@q cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n\t}" ::"r"(dst_s),
      "l"(src), "r"(bytes), "r"(bar_s), "r"(on)
      : "memory");
}
__device__ __forceinline__ void tma_2d_g2s_if_s(uint32_t dst_s, const CUtensorMap* map, int x, int y, uint32_t bar_s, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %5, 0;\n\t"
      "@q cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];\n\t}" ::"r"(dst_s),
      "l"(map), "r"(x), "r"(y), "r"(bar_s), "r"(on)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// predicated forms for code that the whole warp runs and one lane acts on
__device__ __forceinline__ void tc_commit_if_s(uint32_t bar_s, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %1, 0;\n\t"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}" ::"r"(bar_s),
      "r"(on)
      : "memory");
}
__device__ __forceinline__ void mbar_arrive_n_if_s(uint32_t bar_s, uint32_t n, uint32_t on) {
  asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.b32 q, %2, 0;\n\t@q mbarrier.arrive.shared::cta.b64 _, [%0], %1;\n\t}" ::"r"(bar_s),
               "r"(n), "r"(on)
               : "memory");
}
// NK consecutive k-steps of one item issued from one asm block (the issuing thread gets few issue slots,
// so every instruction around an MMA counts).  Descriptors are passed as (lo, hi) words; only lo moves.
// TS: A in tensor memory at a_tmem (+a_step per k-step).  `acc0`: accumulate flag of the first k-step.
// `on`: the whole warp runs the issuer's code with the same values (so that the operands can live in uniform
// registers), and the lane with on != 0 issues.
template <int NK>
__device__ __forceinline__ void tc_mma_ts_burst(uint32_t d_tmem, uint32_t a_tmem, uint32_t a_step, uint32_t b_lo,
                                                uint32_t b_hi, uint32_t b_step, uint32_t idesc, uint32_t acc0, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred p, t, q;\n\t.reg .b64 bd;\n\t.reg .b32 lo, a;\n\t"
      "setp.ne.b32 p, %7, 0;\n\t"
      "setp.ne.b32 q, %8, 0;\n\t"
      "setp.eq.b32 t, 0, 0;\n\t"
      "mov.b64 bd, {%3, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], bd, %6, p;\n\t"
      "add.u32 lo, %3, %5;\n\tadd.u32 a, %1, %2;\n\tmov.b64 bd, {lo, %4};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_tmem), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(acc0), "r"(on)
      : "memory");
  if (NK == 4) {
    asm volatile(
        "{\n\t.reg .pred t, q;\n\t.reg .b64 bd;\n\t.reg .b32 lo, a;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "setp.ne.b32 q, %7, 0;\n\t"
        "mad.lo.u32 lo, %5, 2, %3;\n\tmad.lo.u32 a, %2, 2, %1;\n\tmov.b64 bd, {lo, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
        "add.u32 lo, lo, %5;\n\tadd.u32 a, a, %2;\n\tmov.b64 bd, {lo, %4};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [a], bd, %6, t;\n\t"
        "}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(on)
        : "memory");
  }
}
// SS: A in shared memory, descriptor (a_lo, a_hi), +a_step per k-step.
template <int NK>
__device__ __forceinline__ void tc_mma_ss_burst(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t a_step,
                                                uint32_t b_lo, uint32_t b_hi, uint32_t b_step, uint32_t idesc,
                                                uint32_t acc0, uint32_t on) {
  asm volatile(
      "{\n\t.reg .pred p, t, q;\n\t.reg .b64 ad, bd;\n\t.reg .b32 la, lb;\n\t"
      "setp.ne.b32 p, %8, 0;\n\t"
      "setp.ne.b32 q, %9, 0;\n\t"
      "setp.eq.b32 t, 0, 0;\n\t"
      "mov.b64 ad, {%1, %2};\n\tmov.b64 bd, {%4, %5};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, p;\n\t"
      "add.u32 la, %1, %3;\n\tadd.u32 lb, %4, %6;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
      "}" ::"r"(d_tmem),
      "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(acc0), "r"(on)
      : "memory");
  if (NK == 4) {
    asm volatile(
        "{\n\t.reg .pred t, q;\n\t.reg .b64 ad, bd;\n\t.reg .b32 la, lb;\n\t"
        "setp.eq.b32 t, 0, 0;\n\t"
        "setp.ne.b32 q, %8, 0;\n\t"
        "mad.lo.u32 la, %3, 2, %1;\n\tmad.lo.u32 lb, %6, 2, %4;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
        "add.u32 la, la, %3;\n\tadd.u32 lb, lb, %6;\n\tmov.b64 ad, {la, %2};\n\tmov.b64 bd, {lb, %5};\n\t"
        "@q tcgen05.mma.cta_group::1.kind::f16 [%0], ad, bd, %7, t;\n\t"
        "}" ::"r"(d_tmem),
        "r"(a_lo), "r"(a_hi), "r"(a_step), "r"(b_lo), "r"(b_hi), "r"(b_step), "r"(idesc), "r"(on)
        : "memory");
  }
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

// The slot ring.  Everything that travels through it is one "slot item" of at most kSlotBytes: a quantized
// tile image (codes, scales, zero-points), or one K-half (64 columns, 16 KB) of a 16-bit tile -- the two halves
// of a 16-bit tile are consecutive slot items.  Slot items are numbered in issue order; number `seq` sits in
// slot seq % n_slots and uses phase seq / n_slots of that slot's barriers, so every role finds its own slot
// items without replaying anybody else's.
struct RingPos {
  uint32_t s, par;                               // slot, parity of the full-barrier phase
};
// `recip` = floor(2^32 / n_slots), computed once per kernel: the high product is the quotient or one less, which
// one comparison corrects -- a division by a run-time number is some twenty instructions, and every role does
// one or two at every unit boundary.
__device__ __forceinline__ RingPos ring_pos(uint32_t seq, uint32_t n_slots, uint32_t recip) {
  uint32_t q = __umulhi(seq, recip);
  RingPos p;
  p.s = seq - q * n_slots;
  if (p.s >= n_slots) {
    p.s -= n_slots;
    ++q;
  }
  p.par = q & 1u;
  return p;
}
__device__ __forceinline__ void ring_advance(RingPos& p, uint32_t step, uint32_t n_slots) {
  p.s += step;
  while (p.s >= n_slots) {
    p.s -= n_slots;
    p.par ^= 1u;
  }
}
__device__ __forceinline__ uint32_t slot_items(uint32_t bits) { return bits == 16 ? 2u : 1u; }
// Bounded wait until the weight producer has armed slot item n.  A consumer looks at a slot item's full barrier
// only after this, so it can never mistake an older phase of the slot's barrier for the item's.
template <uint32_t LIM>
__device__ __forceinline__ bool wait_issued(uint32_t n, Ctrl* c, int32_t* status) {
  if (c->issued[n & 1] > n) return true;
  return flag_wait<LIM>(smem_u32(const_cast<uint32_t*>(&c->issued[n & 1])), n, c, status);
}
// Unit i of this CTA's work list (bounded wait until the weight producer has posted it); -1 = no more work,
// -2 = the CTA is aborting.
template <uint32_t LIM>
__device__ __forceinline__ int next_unit(uint32_t i, Ctrl* c, int32_t* status) {
  if (c->sched_n > i) return c->sched_unit[i & 31];
  if (flag_wait<LIM>(smem_u32(const_cast<uint32_t*>(&c->sched_n)), i, c, status)) return c->sched_unit[i & 31];
  return -2;
}
// A unit of the list.  The gate/up list is written by the kernel directly ahead of this one in the stream, possibly
// while this grid is already resident.  Only the two weight producers read it, after they have waited for that
// kernel (grid_dep_sync), so an ordinary cached load sees final data -- what it must not be is a load through the
// non-coherent path, which the compiler may choose for a `const __restrict__` pointer: hence the explicit cache
// operator.  Every other role gets the unit from producer 0 through shared memory (load_desc).
__device__ __forceinline__ Unit load_unit(const Unit* units, int u) {
  const int4* p = reinterpret_cast<const int4*>(units + u);
  const int4 a = __ldca(p), b = __ldca(p + 1);
  Unit un;
  un.seg = a.x;
  un.row_tile = a.y;
  un.tok0 = a.z;
  un.ntok = a.w;
  un.g0 = b.x;
  un.g1 = b.y;
  un.split = b.z;
  un.pad_ = b.w;
  return un;
}
// Unit i of this CTA's work list as producer 0 posted it (after next_unit has returned its index).
__device__ __forceinline__ Unit load_desc(const Ctrl* c, uint32_t i) {
  const uint32_t a_s = smem_u32(&c->desc[i & 15]);
  int4 a, b;
  asm volatile("ld.volatile.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w) : "r"(a_s));
  asm volatile("ld.volatile.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "r"(a_s + 16));
  Unit un;
  un.seg = a.x;
  un.row_tile = a.y;
  un.tok0 = a.z;
  un.ntok = a.w;
  un.g0 = b.x;
  un.g1 = b.y;
  un.split = b.z;
  un.pad_ = b.w;                                 // bitwidths: matrix 0 in bits 0-7, matrix 1 in bits 8-15
  return un;
}
// Bitwidth of a page-table row as the kernel's roles pass it around: the bitwidth, with kPlanesFlag for a block of
// overlaid bit-planes (whose tiles are gathered from up to four places and decoded by their own routines).
constexpr uint32_t kPlanesFlag = 0x40;
template <bool PLANES>
__device__ __forceinline__ uint32_t row_ubits(const DevRow& r) {
  return r.bits | (PLANES && r.valid == 2 ? kPlanesFlag : 0u);
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

// Source of the next item of one matrix of a unit (weight producer).
struct MatSrc {
  uint32_t bits, tb;                              // bitwidth; bytes of a tile image (of a TOP tile for a bit-plane block)
  uint32_t q;                                     // bitwidth a bit-plane block is read at, 0 = an ordinary page
  const char* src;
  const char* b1;                                 // bit-plane blocks: the BIT1 and BIT0 buffers
  const char* b0;
};

// K-half `h` of one row of an item: shared memory -> 32 registers (half2 pairs in K order).
template <int BITS>
__device__ __forceinline__ void decode_item_half(const char* item, int r, int h, __half2* w) {
  const uint4* row_units = reinterpret_cast<const uint4*>(item) + r;
  const __half2 s2 = __half2half2(reinterpret_cast<const __half*>(item + BITS * 2048)[r]);
  const __half2 z2 = __half2half2(reinterpret_cast<const __half*>(item + BITS * 2048 + 256)[r]);
  decode_half<BITS>(row_units, h, s2, z2, w);
}

// predicated arrival (no branch around it)
__device__ __forceinline__ void mbar_arrive_if_s(uint32_t bar_s, bool pred) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %1, 0;\n\t@p mbarrier.arrive.shared::cta.b64 _, [%0];\n\t}" ::"r"(bar_s),
               "r"((uint32_t)pred)
               : "memory");
}

// What a dequantizer warp carries from tile to tile.
struct DqState {
  uint32_t sq;                                   // number of my next slot item
  uint32_t s, par;                               // its ring slot and the parity of its full-barrier phase
  uint32_t a_par;                                // parity of the next "operand slot free" phase of my group
  uint32_t known;                                // the producer of my items has armed every one below this number
};

// The tiles of one unit that fall to this warp's group (`count` of them, `step` slot items apart), all in one code
// format: row r of each tile, both K-halves, into the group's operand slot in tensor memory.  The slot is free once
// the MMAs of the group's previous tile have read it; they ran while the first half was being decoded.  One routine
// per code format, with the tile loop inside: what a decoder computes is stored from the registers it was computed
// in, and nothing about the format is decided per tile.  The per-tile control path is a chain of dependent
// instructions that the decoders of the other groups do not hide, so it is kept as short as it gets.
// UB: bitwidth, with kPlanesFlag for a tile of a bit-plane block.
template <uint32_t UB, uint32_t LIM>
__device__ __forceinline__ bool dq_run(DqState& st, uint32_t count, uint32_t step, uint32_t n_slots, uint32_t wring_s,
                                       int r, bool lane0, uint32_t lane_addr, uint32_t full_s, uint32_t empty_s,
                                       uint32_t a_full_s, uint32_t a_empty_s, Ctrl* c, int32_t* status) {
#pragma unroll 1
  for (; count; --count) {
    // A slot's full barrier is looked at only once the item is known to have been armed (the phase before it has
    // then completed, so the parity cannot be mistaken); the producer is usually several items ahead, and one
    // look at its counter covers them.
    if (st.known <= st.sq) {
      st.known = c->issued[st.sq & 1];
      if (st.known <= st.sq) {
        if (!flag_wait<LIM>(smem_u32(const_cast<uint32_t*>(&c->issued[st.sq & 1])), st.sq, c, status)) return false;
        st.known = st.sq + 1;
      }
    }
    if (!mbar_wait_s<LIM>(full_s + 8 * st.s, st.par, c, status)) return false;
    const uint32_t item_s = wring_s + st.s * kSlotBytes;
    __half2 s2, z2;
    {
      constexpr uint32_t lut = (UB & kPlanesFlag) != 0 ? (uint32_t)kPlaneSlotLut : (UB & 63u) * 2048u;
      uint16_t sv, zv;
      asm volatile("ld.shared.u16 %0, [%1];" : "=h"(sv) : "r"(item_s + lut + 2 * r));
      asm volatile("ld.shared.u16 %0, [%1];" : "=h"(zv) : "r"(item_s + lut + 256 + 2 * r));
      s2 = __half2half2(__ushort_as_half(sv));
      z2 = __half2half2(__ushort_as_half(zv));
    }
    const char* item = reinterpret_cast<const char*>(c) + kCtrlBytes + st.s * kSlotBytes;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      __half2 w[32];
      if constexpr ((UB & kPlanesFlag) != 0) decode_half_planes<(int)(UB & ~kPlanesFlag)>(item, r, h, s2, z2, w);
      else decode_half<(int)UB>(reinterpret_cast<const uint4*>(item) + r, h, s2, z2, w);
      if (h == 0) {
        if (!mbar_wait_s<LIM>(a_empty_s, st.a_par ^ 1, c, status)) return false;
        tc_fence_after();
      } else {
        __syncwarp();
        mbar_arrive_if_s(empty_s + 8 * st.s, lane0);   // this warp has read its rows of the tile
      }
      tmem_st32(lane_addr + h * 32, w);
    }
    // hand the tile over: both stores have landed, then one arrival per warp
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive_if_s(a_full_s, lane0);
    st.a_par ^= 1u;
    st.sq += step;
    st.s += step;
    if (st.s >= n_slots) {                       // step never exceeds the number of slots
      st.s -= n_slots;
      st.par ^= 1u;
    }
  }
  return true;
}

// A warp has stored its share of the SwiGLU rows of a gate/up unit: count it in for the K range of the down
// projection that the unit's FFN rows belong to.  The down kernel, which may already be running on SMs this kernel
// has left, starts a unit when every warp of every gate/up unit it reads has been counted (see the token-tile
// producer); the fence before the count makes the rows visible to it.
__device__ __forceinline__ void signal_rows_done(int32_t* done, int tok0, int row_tile, int n_row_tiles, int dn_splits, int lane) {
  __threadfence();
  __syncwarp();
  if (lane == 0) {
    int sp = 0;                                    // K range sp of the down projection covers [sp * n / splits, (sp + 1) * n / splits)
    while (sp + 1 < dn_splits && ((sp + 1) * n_row_tiles) / dn_splits <= row_tile) ++sp;
    atomicAdd(done + (size_t)tok0 * dn_splits + sp, 1);
  }
}

// Accumulators per matrix of a unit with nb_rows token columns.  The decode kernels give a unit as many partial
// accumulators per matrix as there are issuers per matrix.  For token tiles wider than 32 that fills more than half
// of the accumulator columns: the unit takes both accumulator buffers, and its epilogue cannot overlap the next
// unit's MMAs.  The SHARE instantiations, launched where the epilogue is a large part of a unit (units of at most
// kShortUnitTiles weight tiles), give such a unit fewer accumulators instead, the issuers of a matrix taking turns
// on them tile by tile (the turn word below), and it keeps to one buffer: fine-grained decode, down kernel -12 %,
// gate/up -4 %.  On long units the turns buy nothing, and the code for them costs the gate/up kernel 1 %.
constexpr int kShortUnitTiles = 32;
template <bool SHARE, int NMAT>
__device__ __forceinline__ int unit_accumulators(int npart, int nb_rows, int acol) {
  int npe = npart;
  if (SHARE)
    while (npe > 1 && NMAT * npe * nb_rows > acol / 2) npe >>= 1;
  return npe;
}

// PHASE 0: units of (expert, 128 FFN rows, token tile): gate and up pages -> Ht.
// PHASE 1: units of (expert, 128 hidden rows, token tile, K range): down page -> Y[split].
// PLANES: the instantiation that also reads blocks of overlaid bit-planes; launched only for a layer that holds one
// (the extra code paths cost the ordinary ones instruction-cache room).
// SHORT: the instantiation with the short wait limit (kTestWaitPolls instead of kDefaultWaitPolls), for the test of
// the failure path.  hook: test hook, bit 0 = the token-tile producer stops before its second tile (so that the
// waits on it run out).
template <int PHASE, bool HELP, bool PLANES, bool SHORT, bool SHARE = false>
__global__ void __launch_bounds__(kThreads, 1)
ffn_tc_kernel(const DevRow* __restrict__ rows, const Unit* units, const int32_t* __restrict__ n_units_ptr,
              const __grid_constant__ TmapSet tmaps, int Rpad, int nt_tile, int n_bslots, int n_slots,
              __half* __restrict__ ht, float* __restrict__ y, int H, size_t y_split_stride,
              int32_t* __restrict__ work_counter, int32_t* __restrict__ status, int32_t* done, int dn_splits,
              int ffn_tiles, uint32_t hook) {
  constexpr uint32_t LIM = SHORT ? kTestWaitPolls : kDefaultWaitPolls;
  extern __shared__ __align__(1024) char smem[];
  Ctrl* c = reinterpret_cast<Ctrl*>(smem);
  char* wring = smem + kCtrlBytes;
  char* bslots = wring + n_slots * kSlotBytes;
  const int bslot_bytes = nt_tile * 256;
  constexpr int NMAT = PHASE == 0 ? 2 : 1;
  // the warp number, broadcast: what follows from it (role, group, slot and barrier addresses) is then known to the
  // compiler as the same in all lanes and can be computed and kept in uniform registers
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int n_units = n_units_ptr[PHASE];
  // tensor-memory columns: partial accumulators first ([matrix][partial][nt_tile]), dequantized-operand
  // slots after them.  Partials per matrix: as many as issuers per matrix, while two operand slots still fit.
  constexpr int IPM = kIssuers / NMAT;           // issuers per matrix = dequantizer groups per matrix
  int npart = IPM;
  while (npart > 1 && NMAT * npart * nt_tile + kMaxASlots * 64 > kTmemCols) npart >>= 1;
  // Active issuers per matrix: one per accumulator, except in the gate/up kernel for wide token tiles, where the
  // two issuers of a matrix take turns on its one accumulator (the down kernel's token tiles then leave too few
  // token-tile slots for four issuers: it lost 10 %).
  constexpr bool kSharedAcc = HELP && PHASE == 0;
  const int ipa = kSharedAcc ? IPM : npart;
  const int n_issuers = NMAT * ipa;
  const int acol = NMAT * npart * nt_tile;       // the operand slot of group g sits at acol + 64 * g
  const int G = gridDim.x;
  const uint32_t recip_w = 0xffffffffu / (uint32_t)n_slots, recip_b = 0xffffffffu / (uint32_t)n_bslots;   // see ring_pos

  if (threadIdx.x == 0) {
    for (int i = 0; i < kMaxSlots; ++i) {
      mbar_init(&c->full[i], 1);
      mbar_init(&c->empty[i], 4);                 // four dequantizer warps, or an issuer's commit + 3 arrivals
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
    c->issued[0] = c->issued[1] = 0;
    c->b_issued = 0;
    c->turn[0] = c->turn[1] = c->turn[2] = c->turn[3] = 0;
    c->sched_n = 0;
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
  // grid_dep_sync).  What the kernel directly ahead writes is not: the token rows (the gate/up kernel's
  // token-tile producer waits for the kernel that gathers them, the down kernel's for the completion counters of
  // the gate/up units, one unit at a time) and the gate/up unit list (PHASE 0; the weight producers wait).

  // Units are claimed dynamically: CTA b starts with unit b, every further one comes from the global counter
  // (the weight producer claims, the other roles follow its list).

  if (warp == kWarpCodes || warp == kWarpCodes2) {
    // ---------------- weight producers ----------------
    // Two producer warps share the stream: producer P arms the slot items with number = P mod 2,
    // which (even slot count) always land in the slots = P mod 2, so each keeps the state of its own slots.
    // Producer 0 also claims the units.  The whole warp runs the loop on the same values; lane 0 arms, copies,
    // claims and posts.
    {
      const uint32_t on = lane == 0 ? 1u : 0u;
      const uint32_t P = warp == kWarpCodes ? 0u : 1u;
      uint32_t seq = 0, s = 0;                     // number and slot of the next slot item of the stream
      // A slot is free for slot item seq once the phase seq / n_slots - 1 of its empty barrier has completed
      // (nothing to wait for during the first pass over the ring).
      uint32_t pass = 0;                           // seq / n_slots
      const uint32_t wring_s = smem_u32(wring), full_s = smem_u32(&c->full[0]);
      bool ok = true;
      // The gate/up kernel's unit list is written by the kernel directly ahead of it (the one that gathers
      // the token rows), which may still be running: the producers wait for it before they read a unit, and
      // every other role learns of its first unit from producer 0 only after that.  The down kernel's list is
      // two kernels back and final (see grid_dep_sync), so its producers stream at once.
      if (PHASE == 0) grid_dep_sync();
      // the work list: unit blockIdx.x first, then whatever the global counter hands out
      int u = (int)blockIdx.x < n_units ? (int)blockIdx.x : -1;
      Unit un;
      DevRow rw[NMAT];
      auto fetch_info = [&](int uu) {
        un = load_unit(units, uu);
#pragma unroll
        for (int m = 0; m < NMAT; ++m) rw[m] = rows[un.seg * 3 + (PHASE == 0 ? m : 2)];
      };
      // producer 0 posts a unit: its index, and the unit with the bitwidths of its pages for the other roles
      auto post = [&](uint32_t idx, int uu) {
        if (on) {
          if (uu >= 0) {
            Unit d = un;
            d.pad_ = (int32_t)(row_ubits<PLANES>(rw[0]) | (row_ubits<PLANES>(rw[NMAT - 1]) << 8));
            int4* dp = reinterpret_cast<int4*>(&c->desc[idx & 15]);
            dp[0] = make_int4(d.seg, d.row_tile, d.tok0, d.ntok);
            dp[1] = make_int4(d.g0, d.g1, d.split, d.pad_);
          }
          c->sched_unit[idx & 31] = uu;
          __threadfence_block();
          c->sched_n = idx + 1;
        }
      };
      if (u >= 0) fetch_info(u);
      if (P == 0) post(0u, u);
      for (int i = 0; ok && u >= 0; ++i) {
        int claimed = 0;
        // per matrix of the unit: bitwidth, bytes of a tile image, address of the unit's first tile;
        // consecutive groups of a row tile are consecutive tiles of the page
        MatSrc ms[NMAT];
#pragma unroll
        for (int m = 0; m < NMAT; ++m) {
          const DevRow& row = rw[m];
          const bool planes = PLANES && row.valid == 2;
          ms[m].bits = row.bits;
          ms[m].q = planes ? row.bits : 0u;
          ms[m].tb = planes ? (uint32_t)kPlaneTopTile : (uint32_t)tile_bytes((int)row.bits);
          const size_t tile = (size_t)un.row_tile * (row.cols / kGroup) + un.g0;
          ms[m].src = reinterpret_cast<const char*>(row.codes) + tile * ms[m].tb;
          ms[m].b1 = reinterpret_cast<const char*>(row.bit1) + tile * kPlaneBitTile;
          ms[m].b0 = reinterpret_cast<const char*>(row.bit0) + tile * kPlaneBitTile;
        }
        const int ng = un.g1 - un.g0;
        const int claim_at = ng >> 1;
#pragma unroll 1
        for (int g = 0; ok && g < ng; ++g) {
          // claim the next unit half-way through this one: the answer is back long before it is needed
          if (P == 0 && g == claim_at) {
            int got = 0;
            if (on) got = atomicAdd(work_counter, 1);
            claimed = __shfl_sync(0xffffffffu, got, 0) + G;
          }
#pragma unroll
          for (int m = 0; m < NMAT; ++m) {
            const bool f16 = ms[m].bits == 16;
            const uint32_t q = PLANES ? ms[m].q : 0u;
            // a 16-bit tile goes as two K-halves; of a bit-plane tile read at q bits only the first q bits of every
            // weight leave HBM: the top codes, the planes below them that q needs, the lookup-table state of q
            const uint32_t bytes = f16 ? 16384u : q ? (uint32_t)kPlaneTopCodes + 512u + (q - 2u) * (uint32_t)kPlaneBitTile : ms[m].tb;
            const int nsub = f16 ? 2 : 1;
            const char* src = ms[m].src;
            const char* b1 = ms[m].b1;
            const char* b0 = ms[m].b0;
            ms[m].src += ms[m].tb;
            ms[m].b1 += kPlaneBitTile;
            ms[m].b0 += kPlaneBitTile;
            for (int sub = 0; sub < nsub; ++sub, src += 16384) {
              if ((seq & 1u) == P) {
                if (pass) ok = mbar_wait_s<LIM>(smem_u32(&c->empty[s]), (pass - 1) & 1, c, status);
                if (!ok) break;
                const uint32_t bar_s = full_s + 8 * s;
                mbar_expect_tx_if_s(bar_s, bytes, on);
                const uint32_t slot_s = wring_s + s * kSlotBytes;
                if (q) {
                  bulk_g2s_if_s(slot_s, src, kPlaneTopCodes, bar_s, on);
                  bulk_g2s_if_s(slot_s + kPlaneSlotLut, src + plane_lut_offset((int)q), 512, bar_s, on);
                  if (q >= 3) bulk_g2s_if_s(slot_s + kPlaneSlotBit1, b1, kPlaneBitTile, bar_s, on);
                  if (q == 4) bulk_g2s_if_s(slot_s + kPlaneSlotBit0, b0, kPlaneBitTile, bar_s, on);
                } else {
                  bulk_g2s_if_s(slot_s, src, bytes, bar_s, on);
                }
                if (on) c->issued[P] = seq + 2;        // my next slot item is seq + 2
              }
              ++seq;
              if (++s == (uint32_t)n_slots) {
                s = 0;
                ++pass;
              }
            }
            if (!ok) break;
          }
        }
        if (P == 0) {
          u = claimed < n_units ? claimed : -1;
          if (u >= 0) fetch_info(u);
          post((uint32_t)i + 1, u);
        } else {
          u = next_unit<LIM>((uint32_t)i + 1, c, status);
          if (u >= 0) fetch_info(u);
        }
      }
    }
  } else if (warp == kWarpTokens) {
    // ---------------- token-tile producer ----------------
    // (the whole warp runs the loop on the same values; lane 0 arms and copies)
    {
      const uint32_t on = lane == 0 ? 1u : 0u;
      // The gate/up kernel waits for the kernel ahead of it (which gathers its token rows).  The down kernel does
      // not wait for the gate/up kernel as a whole: its CTAs take the SMs that kernel's CTAs leave one by one, and
      // a unit starts as soon as the gate/up units that write the rows it multiplies have been counted in.
      if (PHASE == 0) grid_dep_sync();
      grid_dep_trigger();
      uint32_t bcount = 0;
      bool ok = true;
      for (int i = 0; ok; ++i) {
        const int u = next_unit<LIM>((uint32_t)i, c, status);
        if (u < 0) break;
        const Unit un = load_desc(c, (uint32_t)i);
        const int nb_rows = (un.ntok + 15) & ~15;
        const CUtensorMap* map = &tmaps.m[(nb_rows >> 4) - 1];
        if (PHASE == 1) {
          // every warp that stores rows of a gate/up unit counts itself in: the four epilogue warps, and the four
          // issuer warps as well where they share the epilogue (that kernel's rule for a wide unit)
          const bool helped = HELP && 2 * nb_rows > nt_tile;
          const int need = (helped ? 8 : 4) * (un.g1 - un.g0);
          const int32_t* flag = done + (size_t)un.tok0 * dn_splits + un.split;
          int seen = 0;
          for (uint32_t n = 0;; ++n) {
            asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(seen) : "l"(flag) : "memory");
            seen = __shfl_sync(0xffffffffu, seen, 0);    // one answer for the warp
            if (seen >= need) break;
            // the gate/up kernel gave up (a wait of its own ran out), or this wait has lasted 2 s
            if (n >= LIM * 64u || *reinterpret_cast<volatile int32_t*>(status) == (int)PW_ERR_TIMEOUT) {
              c->abort_flag = 1;
              atomicMax(status, (int)PW_ERR_TIMEOUT);
              ok = false;
              break;
            }
            __nanosleep(300);
          }
          if (!ok) break;
          asm volatile("fence.proxy.async.global;" ::: "memory");   // the rows were written with ordinary stores; the copies below read them through the async proxy
        }
        for (int g = un.g0; ok && g < un.g1; ++g) {
          if ((hook & 1u) && bcount == 1) {        // test hook: leave the tile unarmed, so that the waits on it run out
            ok = false;
            break;
          }
          // token tile of this group: 16 K-chunks x nb_rows rows x 16 bytes, one 2-D copy
          const int bs = bcount % n_bslots;
          ok = mbar_wait_s<LIM>(smem_u32(&c->b_empty[bs]), ((bcount / n_bslots) & 1) ^ 1, c, status);
          if (!ok) break;
          const uint32_t bf_bar = smem_u32(&c->b_full[bs]);
          mbar_expect_tx_if_s(bf_bar, (uint32_t)(nb_rows * 256), on);
          tma_2d_g2s_if_s(smem_u32(bslots) + (uint32_t)(bs * bslot_bytes), map, un.tok0 * 2, g * 16, bf_bar, on);
          ++bcount;
          if (on) c->b_issued = bcount;
        }
      }
    }
  }
  else if (warp >= kWarpMma && warp < kWarpMma + kIssuers) {
    // ---------------- MMA issuers ----------------
    // Tile k of a matrix (counted over all units) belongs to issuer k mod npart of that matrix, which issues
    // all eight k-steps of it into its own partial accumulator; a quantized tile k is dequantized by the
    // matrix's group k mod IPM, so with npart == IPM every dequantizer group has an issuer of its own.
    // The epilogue adds the partials.
    // The whole warp runs the issuer's code on the same values -- the warp number is broadcast so that the compiler
    // knows it -- and lane 0 issues, commits and arrives: descriptors and addresses computed by a converged warp
    // can stay in uniform registers, which is where the MMA takes its operands from.
    const int iss = warp - kWarpMma;
    const uint32_t on = lane == 0 ? 1u : 0u;
    const int my_m = iss / IPM, my_j = iss % IPM;
    const uint32_t desc_hi = (uint32_t)(make_kmajor_desc(0, 0) >> 32);
    const uint32_t b_lo_base = smem_u32(bslots) >> 4;
    const uint32_t w_lo_base = smem_u32(wring) >> 4;
    const uint32_t af_s = smem_u32(&c->a_full[0]), ae_s = smem_u32(&c->a_empty[0]);
    const uint32_t bf_s = smem_u32(&c->b_full[0]), be_s = smem_u32(&c->b_empty[0]);
    const uint32_t a_base = tmem + acol;
    const uint32_t a_lo_lbo = (2048u >> 4) << 16;                   // A descriptor (16-bit tiles): LBO 2048 B
    // My tiles of one unit (every npart-th group from j0 on): token tile, operand (a 16-bit tile's two halves from
    // the ring, or the operand slot of the group that dequantized the tile), eight MMAs, hand-backs.  One body for
    // both instantiations of the issuer role below.
    uint32_t b_known = 0;                          // token tiles known to have been armed
    // npe: accumulators per matrix of the unit (unit_accumulators); tile k of the matrix goes to accumulator
    // k mod npe.  When that is fewer than the issuers of the matrix, the tiles of an accumulator are issued in
    // order by different issuers: its turn word holds 1 + the number of the last tile whose MMAs are in the pipe.
    // Never more than two issuers share an accumulator (half of the accumulator columns always holds two token
    // tiles of the down kernel, one per matrix of the gate/up kernel), so the only other writer of the word a tile
    // waits on is the issuer of the tile before it -- which writes a later number only after that tile.  The first
    // tile of a unit on an accumulator waits for nobody: the buffer was handed back by the epilogue.
    auto issue_tiles = [&](uint32_t j0, uint32_t ng, uint32_t base, uint32_t W, uint32_t my_bits, uint32_t d_t,
                           uint32_t b_lo_unit, uint32_t b_step, uint32_t idesc, uint32_t& bt, RingPos& bp, uint32_t& sq,
                           RingPos& rp, uint32_t& upar, uint32_t npe) -> bool {
        bool ok = true;
        const bool shared_acc = SHARE ? npe < (uint32_t)ipa : kSharedAcc;
        const uint32_t turn_s = smem_u32(const_cast<uint32_t*>(&c->turn[my_m * npart + (my_j & ((int)npe - 1))]));
        // accumulate onto earlier tiles: after my first tile, and from the start when the accumulator's first tile
        // of this unit is another issuer's
        uint32_t later = j0 >= npe ? 1u : 0u;
        // my MMAs are in the pipe: the accumulator's next tile may follow
        auto release_turn = [&](uint32_t k) {
          if (shared_acc) {
            tc_fence_before();
            // (a maximum, not a store: the issuer that goes first in the next unit may already have written a later
            // number when the one that closes this unit gets here)
            if (on) asm volatile("red.shared.max.u32 [%0], %1;" ::"r"(turn_s), "r"(k + 1) : "memory");
          }
        };
#pragma unroll 1
        for (uint32_t j = j0; ok && j < ng; j += (uint32_t)ipa) {
          const uint32_t tord = base + j;              // number of this tile among the tiles of its matrix
          const bool after = shared_acc && j >= npe;   // another issuer's tile of this unit precedes it on the accumulator
          // the token tile of this group (a tile is looked at only once it is known to have been armed; the
          // producer is usually ahead, and one look at its counter covers the tiles up to it)
          if (b_known <= bt) {
            b_known = c->b_issued;
            if (b_known <= bt) {
              ok = flag_wait<LIM>(smem_u32(const_cast<uint32_t*>(&c->b_issued)), bt, c, status);
              if (!ok) break;
              b_known = bt + 1;
            }
          }
          ok = mbar_wait_s<LIM>(bf_s + 8 * bp.s, bp.par, c, status);
          if (!ok) break;
          const uint32_t b_lo = b_lo_unit + bp.s * (uint32_t)(bslot_bytes >> 4);
          if (my_bits == 16) {
            // each K-half lies in its own slot as a K-major core-matrix image (k-steps 0 .. 3, 4 KB apart)
            RingPos hp = rp;
#pragma unroll 1
            for (uint32_t hh = 0; hh < 2; ++hh) {
              ok = wait_issued<LIM>(sq + hh, c, status) && mbar_wait_s<LIM>(smem_u32(&c->full[hp.s]), hp.par, c, status);
              if (ok && after && hh == 0) ok = flag_wait<LIM>(turn_s, tord - npe, c, status);
              if (!ok) break;
              tc_fence_after();
              const uint32_t a_lo = (w_lo_base + hp.s * (kSlotBytes >> 4)) | a_lo_lbo;
              tc_mma_ss_burst<4>(d_t, a_lo, desc_hi, 256, b_lo + 4 * hh * b_step, desc_hi, b_step, idesc, later | hh, on);
              if (hh == 1) release_turn(tord);
              mbar_arrive_n_if_s(smem_u32(&c->empty[hp.s]), 3, on);   // with the commit: the four arrivals of the slot's phase
              tc_commit_if_s(smem_u32(&c->empty[hp.s]), on);
              ring_advance(hp, 1, (uint32_t)n_slots);
            }
            if (!ok) break;
            sq += (uint32_t)ipa * W;
            ring_advance(rp, (uint32_t)ipa * W, (uint32_t)n_slots);
          } else {
            // the group that dequantizes this tile, and the parity of this use of its operand slot
            const uint32_t k = base + j;
            const uint32_t grp = NMAT == 2 ? 2u * (uint32_t)my_m + (k & 1u) : (k & 3u);
            const uint32_t use_par = (upar >> grp) & 1u;
            upar ^= 1u << grp;
            const uint32_t f0 = af_s + 8 * grp, e0 = ae_s + 8 * grp;       // barriers of the group's operand slot
            const uint32_t a_t = a_base + grp * 64;
            ok = mbar_wait_s<LIM>(f0, use_par, c, status);
            if (ok && after) ok = flag_wait<LIM>(turn_s, tord - npe, c, status);
            if (!ok) break;
            tc_fence_after();
            // all eight k-steps of the tile, then one commit hands the group's operand slot back
            tc_mma_ts_burst<4>(d_t, a_t, 8, b_lo, desc_hi, b_step, idesc, later, on);
            tc_mma_ts_burst<4>(d_t, a_t + 32, 8, b_lo + 4 * b_step, desc_hi, b_step, idesc, 1u, on);
            release_turn(tord);
            tc_commit_if_s(e0, on);
          }
          tc_commit_if_s(be_s + 8 * bp.s, on);
          later = 1;
          bt += (uint32_t)ipa;
          ring_advance(bp, (uint32_t)ipa, (uint32_t)n_bslots);
        }
        return ok;
    };
    if constexpr (!HELP) {
    if (my_j < ipa) {
      uint32_t seq_unit = 0;                        // slot items before the current unit
      uint32_t base = 0;                            // tiles of one matrix (= token tiles) before the current unit
      uint32_t upar = 0;                            // per group: parity of the next use of its operand slot
      uint32_t ucount = 0;
      // Accumulators: partial (m, j) of a unit sits at buffer base + (m * npart + j) * nb_rows.  A unit whose
      // accumulators fit half of the accumulator columns takes one of two buffers in turn, so that its MMAs
      // overlap the epilogue of the unit before it; a wider unit takes both.
      uint32_t dtoggle = 0, duse0 = 0, duse1 = 0;
      bool ok = true;
      for (int i = 0; ok; ++i, ++ucount) {
        const int u = next_unit<LIM>((uint32_t)i, c, status);
        if (u < 0) break;
        const Unit un = load_desc(c, (uint32_t)i);
        uint32_t ubits[NMAT];
#pragma unroll
        for (int m = 0; m < NMAT; ++m) ubits[m] = ((uint32_t)un.pad_ >> (8 * m)) & 0xffu;
        const uint32_t my_bits = my_m ? ubits[NMAT - 1] : ubits[0];
        // slot items per group of the unit (W) and the offset of my matrix's inside a group
        const uint32_t W = slot_items(ubits[0]) + (NMAT == 2 ? slot_items(ubits[NMAT - 1]) : 0u);
        const uint32_t my_off = my_m ? slot_items(ubits[0]) : 0u;
        const uint32_t ng = (uint32_t)(un.g1 - un.g0);
        const int nb_rows = (un.ntok + 15) & ~15;
        const uint32_t idesc = (1u << 4) | ((uint32_t)(nb_rows >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        // B descriptor: leading byte offset = nb_rows * 16 (field at bit 16), advance 2 * nb_rows k-chunk units per k-step
        const uint32_t b_lo_unit = b_lo_base | ((uint32_t)nb_rows << 16);
        const uint32_t b_step = (uint32_t)(2 * nb_rows);
        // my first tile of the unit and what follows from its number: token-tile slot, ring slot, group
        const uint32_t j0 = ((uint32_t)my_j - base) & (uint32_t)(ipa - 1);
        uint32_t bt = base + j0;                     // token-tile number
        RingPos bp = ring_pos(bt, (uint32_t)n_bslots, recip_b);
        uint32_t sq = seq_unit + j0 * W + my_off;    // first slot item of my tile (16-bit tiles only)
        RingPos rp = ring_pos(sq, (uint32_t)n_slots, recip_w);
        const int npe = unit_accumulators<SHARE, NMAT>(npart, nb_rows, acol);
        const bool wide = NMAT * npe * nb_rows > acol / 2;
        const uint32_t dbuf = wide ? 0u : dtoggle;
        if (!wide) dtoggle ^= 1u;
        const uint32_t d_t = tmem + dbuf * (uint32_t)(acol / 2) + (uint32_t)((my_m * npe + (my_j & (npe - 1))) * nb_rows);
        // the epilogue has drained the buffer(s) this unit accumulates into
        if (wide || dbuf == 0) ok = mbar_wait_s<LIM>(smem_u32(&c->d_empty[0]), (duse0 & 1) ^ 1, c, status);
        if (ok && (wide || dbuf == 1)) ok = mbar_wait_s<LIM>(smem_u32(&c->d_empty[1]), (duse1 & 1) ^ 1, c, status);
        if (!ok) break;
        tc_fence_after();
        ok = issue_tiles(j0, ng, base, W, my_bits, d_t, b_lo_unit, b_step, idesc, bt, bp, sq, rp, upar, (uint32_t)npe);
        if (ok) {
          if (wide || dbuf == 0) {
            tc_commit_if_s(smem_u32(&c->d_full[0]), on);
            ++duse0;
          }
          if (wide || dbuf == 1) {
            tc_commit_if_s(smem_u32(&c->d_full[1]), on);
            ++duse1;
          }
        }
        base += ng;
        seq_unit += ng * W;
      }
    }
    } else {
    // Wide token tiles leave no room for a second accumulator buffer, so the epilogue of a unit is not
    // overlapped: here the four issuer warps share it with the four epilogue warps (they take the upper
    // half of the token columns of their lane quarter), lane 0 of the warps with an accumulator of their own
    // issuing the unit's MMAs first.  Every lane tracks the per-unit state; only lane 0 uses the issuing part.
    const bool issuing = my_j < ipa;
    const int hq = warp & 3;
    const int hr = hq * 32 + lane;
    const uint32_t hlane_addr = tmem + ((uint32_t)(hq * 32) << 16);
    {
      uint32_t seq_unit = 0;                        // slot items before the current unit
      uint32_t base = 0;                            // tiles of one matrix (= token tiles) before the current unit
      uint32_t upar = 0;                            // per group: parity of the next use of its operand slot
      uint32_t ucount = 0;
      uint32_t dtoggle = 0, duse0 = 0, duse1 = 0;
      bool ok = true;
      for (int i = 0; ok; ++i, ++ucount) {
        const int u = next_unit<LIM>((uint32_t)i, c, status);
        if (u < 0) break;
        const Unit un = load_desc(c, (uint32_t)i);
        uint32_t ubits[NMAT];
#pragma unroll
        for (int m = 0; m < NMAT; ++m) ubits[m] = ((uint32_t)un.pad_ >> (8 * m)) & 0xffu;
        const uint32_t my_bits = my_m ? ubits[NMAT - 1] : ubits[0];
        // slot items per group of the unit (W) and the offset of my matrix's inside a group
        const uint32_t W = slot_items(ubits[0]) + (NMAT == 2 ? slot_items(ubits[NMAT - 1]) : 0u);
        const uint32_t my_off = my_m ? slot_items(ubits[0]) : 0u;
        const uint32_t ng = (uint32_t)(un.g1 - un.g0);
        const int nb_rows = (un.ntok + 15) & ~15;
        const uint32_t idesc = (1u << 4) | ((uint32_t)(nb_rows >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        // B descriptor: leading byte offset = nb_rows * 16 (field at bit 16), advance 2 * nb_rows k-chunk units per k-step
        const uint32_t b_lo_unit = b_lo_base | ((uint32_t)nb_rows << 16);
        const uint32_t b_step = (uint32_t)(2 * nb_rows);
        // my first tile of the unit and what follows from its number: token-tile slot, ring slot, group
        const uint32_t j0 = ((uint32_t)my_j - base) & (uint32_t)(ipa - 1);
        uint32_t bt = base + j0;                     // token-tile number
        RingPos bp = ring_pos(bt, (uint32_t)n_bslots, recip_b);
        uint32_t sq = seq_unit + j0 * W + my_off;    // first slot item of my tile (16-bit tiles only)
        RingPos rp = ring_pos(sq, (uint32_t)n_slots, recip_w);
        const int npe = unit_accumulators<SHARE, NMAT>(npart, nb_rows, acol);
        const bool wide = NMAT * npe * nb_rows > acol / 2;
        const uint32_t dbuf = wide ? 0u : dtoggle;
        if (!wide) dtoggle ^= 1u;
        const uint32_t d_t = tmem + dbuf * (uint32_t)(acol / 2) + (uint32_t)((my_m * npe + (my_j & (npe - 1))) * nb_rows);
        if (issuing) {
          do {
        // the epilogue has drained the buffer(s) this unit accumulates into
        if (wide || dbuf == 0) ok = mbar_wait_s<LIM>(smem_u32(&c->d_empty[0]), (duse0 & 1) ^ 1, c, status);
        if (ok && (wide || dbuf == 1)) ok = mbar_wait_s<LIM>(smem_u32(&c->d_empty[1]), (duse1 & 1) ^ 1, c, status);
        if (!ok) break;
        tc_fence_after();
        ok = issue_tiles(j0, ng, base, W, my_bits, d_t, b_lo_unit, b_step, idesc, bt, bp, sq, rp, upar, (uint32_t)npe);
            if (ok) {
              if (wide || dbuf == 0) tc_commit_if_s(smem_u32(&c->d_full[0]), on);
              if (wide || dbuf == 1) tc_commit_if_s(smem_u32(&c->d_full[1]), on);
            }
          } while (false);
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        const uint32_t par0 = duse0 & 1u, par1 = duse1 & 1u;     // phases of d_full this unit completes
        if (wide || dbuf == 0) ++duse0;
        if (wide || dbuf == 1) ++duse1;
        // every issuer warp sees every phase of the accumulator barriers, also of the narrow units it has no
        // part in: it must not run ahead of the epilogue by more than the phase parity can tell apart
        if (wide || dbuf == 0) ok = mbar_wait_s<LIM>(smem_u32(&c->d_full[0]), par0, c, status);
        if (ok && (wide || dbuf == 1)) ok = mbar_wait_s<LIM>(smem_u32(&c->d_full[1]), par1, c, status);
        if (!ok) break;
        if (wide) {
          tc_fence_after();
          const uint32_t p0 = base & (uint32_t)(npe - 1), nq = ng < (uint32_t)npe ? ng : (uint32_t)npe;
          const int row = un.row_tile * kTileRows + hr;
          const int half = ((nb_rows / 16 + 1) / 2) * 16;         // the epilogue warps take [0, half)
          for (int c0 = half; c0 < nb_rows; c0 += 16) {
            float a[16], b[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) a[j] = b[j] = 0.0f;
            for (uint32_t q = 0; q < nq; ++q) {
              const int p = (int)((p0 + q) & (uint32_t)(npe - 1));
              float t[16];
              tmem_ld16(hlane_addr + p * nb_rows + c0, t);
              tmem_wait_ld();
#pragma unroll
              for (int j = 0; j < 16; ++j) a[j] = __fadd_rn(a[j], t[j]);
              if (PHASE == 0) {
                tmem_ld16(hlane_addr + (npe + p) * nb_rows + c0, t);
                tmem_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) b[j] = __fadd_rn(b[j], t[j]);
              }
            }
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int nn = c0 + j;
              if (nn < un.ntok) {
                if (PHASE == 0) {
                  const float hval = __fmul_rn(__fdividef(a[j], __fadd_rn(1.0f, __expf(-a[j]))), b[j]);
                  ht[((size_t)(row >> 3) * Rpad + un.tok0 + nn) * 8 + (row & 7)] = __float2half_rn(hval);
                } else {
                  y[(size_t)un.split * y_split_stride + (size_t)(un.tok0 + nn) * H + row] = a[j];
                }
              }
            }
          }
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&c->d_empty[0]);
            mbar_arrive(&c->d_empty[1]);
          }
          if (PHASE == 0) signal_rows_done(done, un.tok0, un.row_tile, ffn_tiles, dn_splits, lane);
        }
        base += ng;
        seq_unit += ng * W;
      }
    }
    }
  } else if (warp < kDqWarps) {    // ---------------- dequantize ----------------
    // Four groups of four warps, each taking every other quantized item of one matrix (every fourth when
    // the unit has a single matrix; an item = one group of one matrix).  Warp q of a group owns rows (= TMEM lanes) 32q .. 32q+31 of the item, one row per
    // thread.  Each group has one operand slot (64 columns: both K-halves of an item): it stores the two halves
    // as it decodes them and hands the slot over once per item; while the issuer's eight MMAs read it, the group
    // decodes the first half of its next item in registers.
    const int grp = warp >> 2, q = warp & 3;
    const int r = q * 32 + lane;                     // weight row inside the tile = TMEM lane
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16) + acol + grp * 64;
    const int qm = NMAT == 2 ? grp >> 1 : 0;         // the matrix this group serves
    const uint32_t gsub = NMAT == 2 ? (uint32_t)(grp & 1) : (uint32_t)grp;   // which of that matrix's groups
    constexpr uint32_t kStride = NMAT == 2 ? 2 : 4;  // groups per matrix = distance between my tiles
    uint32_t seq_unit = 0;                           // slot items before the current unit
    uint32_t base = 0;                               // tiles of one matrix before the current unit
    DqState st;
    st.sq = st.s = st.par = st.a_par = st.known = 0;
    const uint32_t wring_s = smem_u32(wring);
    const uint32_t full_s = smem_u32(&c->full[0]), empty_s = smem_u32(&c->empty[0]);
    const uint32_t a_full_s = smem_u32(&c->a_full[grp]), a_empty_s = smem_u32(&c->a_empty[grp]);
    const bool lane0 = lane == 0;
    bool ok = true;
    for (int i = 0; ok; ++i) {
      const int u = next_unit<LIM>((uint32_t)i, c, status);
      if (u < 0) break;
      const Unit un = load_desc(c, (uint32_t)i);
      uint32_t ubits[NMAT];
#pragma unroll
      for (int m = 0; m < NMAT; ++m) ubits[m] = ((uint32_t)un.pad_ >> (8 * m)) & 0xffu;
      const uint32_t bits = qm ? ubits[NMAT - 1] : ubits[0];
      const uint32_t W = slot_items(ubits[0]) + (NMAT == 2 ? slot_items(ubits[NMAT - 1]) : 0u);
      const uint32_t ng = (uint32_t)(un.g1 - un.g0);
      // Tile k of a matrix (counted over all units) goes to that matrix's group k mod kStride: my first one
      // in this unit is group j0, then every kStride-th.
      const uint32_t j0 = (gsub - base) & (kStride - 1);
      if (bits != 16 && j0 < ng) {                   // the MMA reads 16-bit tiles straight from shared memory
        const uint32_t count = (ng - j0 + kStride - 1) / kStride;
        const uint32_t step = kStride * W;
        st.sq = seq_unit + j0 * W + (qm ? slot_items(ubits[0]) : 0u);
        const RingPos rp = ring_pos(st.sq, (uint32_t)n_slots, recip_w);
        st.s = rp.s;
        st.par = rp.par;
        st.known = 0;                                // my items of this unit may be another producer's than before
#define PW_DQ_RUN(UB) \
  dq_run<UB, LIM>(st, count, step, (uint32_t)n_slots, wring_s, r, lane0, lane_addr, full_s, empty_s, a_full_s, a_empty_s, c, status)
        switch (bits) {
          case 8: ok = PW_DQ_RUN(8); break;
          case 4: ok = PW_DQ_RUN(4); break;
          case 3: ok = PW_DQ_RUN(3); break;
          case 2: ok = PW_DQ_RUN(2); break;
          default:
            if constexpr (PLANES) {
              if (bits == (kPlanesFlag | 4)) ok = PW_DQ_RUN(kPlanesFlag | 4);
              else if (bits == (kPlanesFlag | 3)) ok = PW_DQ_RUN(kPlanesFlag | 3);
              else ok = PW_DQ_RUN(kPlanesFlag | 2);
            }
            break;
        }
#undef PW_DQ_RUN
      }
      base += ng;
      seq_unit += ng * W;
    }
  } else if (warp >= kWarpEpi) {
    // ---------------- epilogue ----------------
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(q * 32) << 16);
    uint32_t ucount = 0, base = 0;                   // base: tiles of one matrix before the current unit
    uint32_t dtoggle = 0, duse0 = 0, duse1 = 0;      // accumulator buffers: the issuers' rule, replayed
    bool ok = true;
    for (int i = 0; ok; ++i, ++ucount) {
      const int u = next_unit<LIM>((uint32_t)i, c, status);
      if (u < 0) break;
      const Unit un = load_desc(c, (uint32_t)i);
      const int nb_rows = (un.ntok + 15) & ~15;
      const int npe = unit_accumulators<SHARE, NMAT>(npart, nb_rows, acol);    // the issuers' rule
      const bool wide = NMAT * npe * nb_rows > acol / 2;
      const uint32_t dbuf = wide ? 0u : dtoggle;
      if (!wide) dtoggle ^= 1u;
      if (wide || dbuf == 0) ok = mbar_wait_s<LIM>(smem_u32(&c->d_full[0]), duse0 & 1, c, status);
      if (ok && (wide || dbuf == 1)) ok = mbar_wait_s<LIM>(smem_u32(&c->d_full[1]), duse1 & 1, c, status);
      if (!ok) break;
      tc_fence_after();
      const int row = un.row_tile * kTileRows + r;
      const uint32_t dbase = lane_addr + dbuf * (uint32_t)(acol / 2);
      // Partial accumulator p holds the tiles base + j with (base + j) mod npart == p.  They are added starting
      // with the one that holds the unit's first tile, so that the order of the sum depends on the unit alone
      // and not on how many tiles this CTA has seen before it (units are claimed in a different order from run
      // to run): a forward call repeats bit for bit.
      const uint32_t ng = (uint32_t)(un.g1 - un.g0);
      const uint32_t p0 = base & (uint32_t)(npe - 1), nq = ng < (uint32_t)npe ? ng : (uint32_t)npe;
      base += ng;
      // with helpers, the issuer warps take the upper half of the token columns of a wide unit
      const int c_end = HELP && wide ? ((nb_rows / 16 + 1) / 2) * 16 : nb_rows;
      for (int c0 = 0; c0 < c_end; c0 += 16) {
        float a[16], b[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) a[j] = b[j] = 0.0f;
        for (uint32_t q = 0; q < nq; ++q) {            // add the issuers' partial sums, in the unit's tile order
          const int p = (int)((p0 + q) & (uint32_t)(npe - 1));
          float t[16];
          tmem_ld16(dbase + p * nb_rows + c0, t);
          tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 16; ++j) a[j] = __fadd_rn(a[j], t[j]);
          if (PHASE == 0) {
            tmem_ld16(dbase + (npe + p) * nb_rows + c0, t);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 16; ++j) b[j] = __fadd_rn(b[j], t[j]);
          }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int nn = c0 + j;
          if (nn < un.ntok) {
            if (PHASE == 0) {
              // SwiGLU: silu(gate) * up; the result is rounded to fp16, so the fast exponential and
              // division (relative error ~1e-6) change nothing that survives the rounding
              const float hval = __fmul_rn(__fdividef(a[j], __fadd_rn(1.0f, __expf(-a[j]))), b[j]);
              ht[((size_t)(row >> 3) * Rpad + un.tok0 + nn) * 8 + (row & 7)] = __float2half_rn(hval);
            } else {
              y[(size_t)un.split * y_split_stride + (size_t)(un.tok0 + nn) * H + row] = a[j];
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        // (a narrow unit has no helpers: this warp arrives for the issuer warp of its lane quarter as well)
        const uint32_t n_arr = HELP && !wide ? 2u : 1u;
        if (wide || dbuf == 0) mbar_arrive_n(&c->d_empty[0], n_arr);
        if (wide || dbuf == 1) mbar_arrive_n(&c->d_empty[1], n_arr);
      }
      // (after the accumulators have been handed back: the fence in there waits for the stores above)
      if (PHASE == 0) signal_rows_done(done, un.tok0, un.row_tile, ffn_tiles, dn_splits, lane);
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

typedef void (*FfnKernel)(const DevRow*, const Unit*, const int32_t*, const TmapSet, int, int, int, int, __half*, float*, int, size_t,
                          int32_t*, int32_t*, int32_t*, int, int, uint32_t);
// share: the instantiation whose wide units take fewer accumulators (decode kernels only)
static FfnKernel ffn_kernel_of(int phase, int help, int planes, int share = 0) {
  static const FfnKernel shared[4] = {ffn_tc_kernel<0, false, false, false, true>, ffn_tc_kernel<1, false, false, false, true>,
                                      ffn_tc_kernel<0, false, true, false, true>, ffn_tc_kernel<1, false, true, false, true>};
  if (share && !help) return shared[phase + 2 * planes];
  static const FfnKernel tab[8] = {
      ffn_tc_kernel<0, false, false, false>, ffn_tc_kernel<1, false, false, false>, ffn_tc_kernel<0, true, false, false>,
      ffn_tc_kernel<1, true, false, false>,  ffn_tc_kernel<0, false, true, false>,  ffn_tc_kernel<1, false, true, false>,
      ffn_tc_kernel<0, true, true, false>,   ffn_tc_kernel<1, true, true, false>};
  return tab[phase + 2 * help + 4 * planes];
}
// the gate/up kernel with the short wait limit (narrow token tiles, ordinary pages): what the failure-path test runs
static FfnKernel ffn_kernel_short() { return ffn_tc_kernel<0, false, false, true>; }

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
  for (int i = 0; i < 4; ++i)
    PW_CUDA_OK(cudaFuncSetAttribute(ffn_kernel_of(i & 1, 0, (i >> 1) & 1, 1), cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kMaxDynSmem));
  PW_CUDA_OK(cudaFuncSetAttribute(ffn_kernel_short(), cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
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

static bool planes_layer(const pw_ctx* ctx, int layer) {     // does the layer hold a bit-plane block?
  for (int e = 0; e < ctx->ws.S; ++e)
    for (int u = 0; u < 3; ++u)
      if (ctx->host_rows[row_index(ctx, layer, e, u)].page.layout == PW_LAYOUT_PLANES) return true;
  return false;
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
    // every issuer of a matrix works on a token tile of its own, one more is on its way -- fewer when the tiles are
    // so wide that the weight ring would fall below six slots
    const int ipa = phase == 0 && nt_tile > 64 ? kIssuers / nmat : npart;   // active issuers per matrix (the kernel's rule)
    int nb = ipa + 1 > kMaxBSlots ? kMaxBSlots : ipa + 1;
    int ns = 0;
    for (;; --nb) {
      ns = (kMaxDynSmem - kCtrlBytes - nb * bslot_bytes) / kSlotBytes;
      if (ns > kMaxSlots) ns = kMaxSlots;
      ns &= ~1;                                  // an even number of slots: one set per producer
      if (ns >= 6 || nb <= npart + 1) break;
    }
    n_bslots[phase] = nb;
    if (ns < 6) return PW_ERR_NOMEM;             // the dequantizers advance up to six slot items at a time
    n_slots[phase] = ns;
    smem[phase] = kCtrlBytes + ns * kSlotBytes + n_bslots[phase] * bslot_bytes;
  }
  const int R = T * k + c.n_shared * T;
  const DevRow* rows = reinterpret_cast<const DevRow*>(b + w.table) + (size_t)layer * w.S * 3;
  int32_t* status = reinterpret_cast<int32_t*>(b + w.status);
  const int32_t* n_units = reinterpret_cast<const int32_t*>(b + w.n_units);
  int32_t* work_counter = reinterpret_cast<int32_t*>(b + w.counter);   // [0] gate/up, [1] down; zeroed by the permute kernel
  timing_mark(ctx, PW_K_FFN_GATE_UP, s);
  // token tiles of 128 leave no second accumulator buffer: the variant whose issuer warps share the epilogue
  const bool help = nt_tile > 64;
  const bool planes = planes_layer(ctx, layer);
  // a context with a lowered wait limit (pw_debug_set_wait) runs the gate/up kernel's short-limit instantiation
  const bool short_wait = ctx->wait_polls != 0 && !help && !planes;
  // short units (few weight tiles between two epilogues): the instantiations that keep wide units to one buffer
  const int share_gu = 2 * (c.hidden / kGroup) <= kShortUnitTiles;
  const int share_dn = (c.ffn / kGroup + ksplit - 1) / ksplit <= kShortUnitTiles;
  PW_CUDA_OK(launch_dependent(short_wait ? ffn_kernel_short() : ffn_kernel_of(0, help, planes, share_gu), dim3(ctx->num_sms),
                              dim3(kThreads), (size_t)smem[0], s, rows,
                              reinterpret_cast<const Unit*>(b + w.units_gu), n_units, st->xt, w.Rpad, nt_tile, n_bslots[0],
                              n_slots[0], reinterpret_cast<__half*>(b + w.ht), (float*)nullptr, c.hidden, (size_t)0,
                              work_counter, status, reinterpret_cast<int32_t*>(b + w.done), ksplit, c.ffn / kTileRows, ctx->test_hook));
  timing_mark(ctx, PW_K_FFN_DOWN, s);
  PW_CUDA_OK(launch_dependent(ffn_kernel_of(1, help, planes, share_dn), dim3(ctx->num_sms), dim3(kThreads), (size_t)smem[1], s, rows,
                              reinterpret_cast<const Unit*>(b + w.units_dn), n_units, st->ht, w.Rpad, nt_tile, n_bslots[1],
                              n_slots[1], (__half*)nullptr, reinterpret_cast<float*>(b + w.y), c.hidden,
                              (size_t)R * c.hidden, work_counter + 1, status, reinterpret_cast<int32_t*>(b + w.done), ksplit, c.ffn / kTileRows, 0u));
  ctx->launches += 2;
  PW_CUDA_OK(cudaGetLastError());
  return PW_OK;
}

}  // namespace pw
