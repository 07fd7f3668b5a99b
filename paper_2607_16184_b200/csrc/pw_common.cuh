// Shared declarations of the library's translation units (host object, device table row,
// workspace map, launch helpers).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/pw.h"

namespace pw {

constexpr int kGroup = 128;      // weights per quantization group
constexpr int kTileRows = 128;   // rows of one page tile
constexpr int kPadRows = 256;    // zero rows appended to the token-major operand buffers
constexpr int kNormSplit = 8;    // observation taps: the squares of an operand row are summed in this many slices

// One row of the device-resident page table (48 bytes).
struct DevRow {
  const void* codes;             // the TILED page buffer (tile images: codes, scales, zero-points)
  uint32_t rows, cols;
  uint32_t bits;
  uint32_t valid;                // 0 = unpublished, 1 = TILED page, 2 = overlaid bit-planes (codes = TOP buffer)
  const void* bit1;              // bit-plane buffers of a PLANES block (null where detached)
  const void* bit0;
  uint64_t reserved;
};
static_assert(sizeof(DevRow) == 48, "DevRow layout");

// One unit of work of the tensor-core FFN kernels.
struct Unit {
  int32_t seg;       // segment index: routed expert e, or E + s for shared expert s
  int32_t row_tile;  // 128-row tile of the weight block
  int32_t tok0;      // first operand row of the token tile (absolute row in Xt / Ht)
  int32_t ntok;      // valid tokens in the tile
  int32_t g0, g1;    // group range [g0, g1) of the contraction
  int32_t split;     // split-K slot the partial result goes to
  int32_t pad_;
};

// Offsets (bytes) of everything that lives in the caller's workspace.
struct WsMap {
  size_t status;      // int32[64]
  size_t counter;     // int32[64]  dynamic work counters
  size_t table;       // DevRow[n_layers * S * 3]
  size_t topk_ids;    // int32[Tmax * kmax]
  size_t gates;       // float[Tmax * kmax]
  size_t counts;      // int32[S]
  size_t offsets;     // int32[S + 1]   (absolute operand rows; shared segments follow the routed pairs)
  size_t perm;        // int32[Pmax]
  size_t inv_perm;    // int32[Pmax]
  size_t row_token;   // int32[Rpad]    operand row -> token (-1 for padding)
  size_t seg_order;   // int32[S]
  size_t tile_tab;    // int2[2][max_tiles]: (segment, token tile of the segment) of every token tile of the two unit lists
  size_t units_gu;    // Unit[max_units]
  size_t units_dn;    // Unit[max_units]
  size_t n_units;     // int32[4]
  size_t done;        // int32[Rmax * 8]: gate/up units finished, per (first operand row of a token tile, K range of the down projection)
  size_t xt;          // fp16 operand rows, k-chunk major: [H/8][Rpad][8]
  size_t ht;          // fp16 SwiGLU output,  k-chunk major: [F/8][Rpad][8]
  size_t y;           // float [y_slots][H]  split-K partial outputs of the down projection
  size_t io_hidden;   // fp16 [Tmax][H]   device staging of pw_moe_forward_host
  size_t io_logits;   // float [Tmax][E]
  size_t io_out;      // float [Tmax][H]
  size_t obs_part;    // float [kNormSplit][2][Rpad]  partial squared norms of the operand rows (observation taps)
  size_t total;
  // derived sizes
  int S;              // segments = E + n_shared
  int Rmax;           // max operand rows = Tmax*kmax + n_shared*Tmax
  int Rpad;           // Rmax + kPadRows
  int max_units;
  int max_tiles;
  size_t y_slots;     // rows of the y buffer (split * R must fit)
};

WsMap make_wsmap(const pw_config& c);

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace pw

struct pw_page_table {
  pw_ctx* owner;
};

namespace pw {
// Residency record of the page of one page-table row at one bitwidth (Sec. 3.1: GPU-resident, CPU-resident
// or in transfer).  A transfer is a copy enqueued on a stream plus an event behind it; the record moves on
// to `heading` when a later call finds the event complete.
constexpr int kBitLevels = 7;                      // pages at 16, 8, 4, 3, 2 bits; planes 3 and 4 of a bit-plane block
struct PageRecord {
  uint8_t state;        // PW_STATE_*
  uint8_t heading;      // state the page reaches when its transfer has finished
  void* dev;            // device buffer (GPU-resident, or source / target of the transfer)
  void* host;           // host buffer (CPU-resident, or target / source of the transfer)
  cudaEvent_t ev;       // created on first use
};
inline int bit_level(int bits) { return bits == 16 ? 0 : bits == 8 ? 1 : bits == 4 ? 2 : bits == 3 ? 3 : bits == 2 ? 4 : -1; }
// record of the plane that reading at `plane` bits adds to reading at plane - 1 bits (3: BIT1, 4: BIT0)
inline int plane_level(int plane) { return plane == 3 ? 5 : plane == 4 ? 6 : -1; }
}  // namespace pw

struct pw_ctx {
  pw_config cfg;
  pw::WsMap ws;
  char* base;                     // cfg.workspace
  pw_page_table table_handle;
  pw_table_entry* host_rows;      // mirror of the committed table
  uint8_t* host_valid;
  uint64_t epoch;
  size_t n_rows;                  // rows of the table = n_layers * (n_experts + n_shared) * 3
  uint64_t launches;
  int last_T, last_k;
  int num_sms;
  void* tc_state;                 // tensor-core path state (set up lazily)
  uint32_t wait_polls;            // limit of the device-side waits in polls of 20 us (0 = the default, 2 s)
  uint32_t test_hook;             // device-side test hooks (pw_debug_set_wait)
  // optional per-kernel timing: a ring of call slots, PW_NUM_KERNELS + 1 events each
  static constexpr int kTimingSlots = 256;
  bool timing_on;
  cudaEvent_t* timing_ev;         // [kTimingSlots][PW_NUM_KERNELS + 1], created on first enable
  bool timing_busy[kTimingSlots];
  int timing_cur;                 // slot of the forward call being enqueued
  uint64_t timing_calls;
  double timing_ms[PW_NUM_KERNELS];
  float* obs_acc;                 // observation accumulators of the caller (device), or null: taps off
  pw::PageRecord* records;        // [rows of the table][kBitLevels]
};

namespace pw {
inline size_t row_index(const pw_ctx* ctx, int layer, int expert, int kind) {
  return ((size_t)layer * ctx->ws.S + expert) * 3 + kind;
}
}  // namespace pw

#define PW_CUDA_OK(expr)                                   \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) return PW_ERR_CUDA;            \
  } while (0)

namespace pw {

// entry points of the other translation units
pw_status launch_route(pw_ctx* ctx, int layer, const void* hidden, const float* logits, int T, int k, int nt_tile,
                       int ksplit, cudaStream_t s);
pw_status launch_combine(pw_ctx* ctx, int T, int k, int ksplit, float* out, cudaStream_t s);
pw_status launch_observe(pw_ctx* ctx, int layer, int T, int k, cudaStream_t s);
// residency records: the state of (row, bits) after looking at its transfer event; registration of a page
// that is being committed (PW_ERR_STATE if the record says that page is away or on its way)
int residency_poll(pw_ctx* ctx, size_t row, int bits);
pw_status residency_check_commit(pw_ctx* ctx, size_t row, const pw_page& page);
void residency_note_commit(pw_ctx* ctx, size_t row, const pw_page& page);
void residency_teardown(pw_ctx* ctx);
// the same for a row that is committed to a block of bit-planes read at page.bits: the planes 3 .. bits
pw_status residency_check_commit_planes(pw_ctx* ctx, size_t row, const pw_page& page);
void residency_note_commit_planes(pw_ctx* ctx, size_t row, const pw_page& page);
pw_status launch_ffn_simt(pw_ctx* ctx, int layer, int T, int k, cudaStream_t s);
pw_status launch_ffn_tensor(pw_ctx* ctx, int layer, int T, int k, int nt_tile, int ksplit, cudaStream_t s);
int tensor_token_tile(const pw_ctx* ctx, int T, int k);
void tc_teardown(pw_ctx* ctx);
// records timing event `i` of the current forward call (no-op unless timing is enabled)
void timing_mark(pw_ctx* ctx, int i, cudaStream_t s);


// ---- programmatic dependent launch -------------------------------------------------------------
// The kernels of one forward call run back to back on one stream.  Each is launched with programmatic
// stream serialization: its CTAs may be placed on an SM, and start, while the kernel before it is still
// finishing elsewhere.  grid_dep_sync() returns once the kernel before this one has completed and its writes
// are visible; a thread calls it before it reads anything that kernel wrote.  grid_dep_trigger() lets the
// kernel after this one be placed as soon as SMs free up; a kernel calls it only after its own
// grid_dep_sync(), so "my CTA has been placed" implies that every kernel two or more steps back in the chain
// has completed.  That is what allows the down kernel to start streaming weight pages at once (its unit list,
// the zeroed completion counters and the page-table rows are written two steps back or earlier); the gate/up
// kernel's unit list is written one step back, so its weight producers wait as well.  The down kernel is the
// one exception to "sync, then trigger": it never waits for the gate/up kernel as a whole but, unit by unit,
// for the completion counters that kernel's epilogue raises (WsMap::done), and the kernel after it reads
// nothing of the gate/up kernel's and waits for the down kernel before it reads anything at all.
// With the timing events between the kernels the attribute has no effect.
// Pointer qualifiers follow from this: `const __restrict__` (which allows non-coherent loads) only on data that
// is final when the kernel is placed -- pages, page-table rows, anything written two or more kernels back; a
// buffer that the kernel directly ahead writes is passed as a plain pointer and read after grid_dep_sync().
__device__ __forceinline__ void grid_dep_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_sync() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace pw
