/*
 * pw.h -- C ABI of the paged-weight MoE hot path for NVIDIA B200 (sm_100a).
 *
 * The library executes one Mixture-of-Experts layer whose expert weight matrices
 * ("linear-blocks", one row of the paper's weight page table each, Sec. 3.1) are
 * resident in GPU memory as weight pages of differing, runtime-changing bitwidths,
 * and lowers the bitwidth of a page at runtime (the "offload" direction of
 * Sec. 3.1 / 3.3).  The paper's pages are Any-Precision bit-planes plus a centroid
 * table; here a page is a group-wise uniform code (group of 128 weights along the
 * input dimension, fp16 scale, fp16 zero-point = the value code 0 decodes to):
 *
 *      weight = fp16( code * scale + zero_point ),   code in [0, 2^bits - 1]
 *
 * General rules
 *   - Plain C.  Every call returns a pw_status; nothing throws, traps or hangs.
 *   - "device" pointers are CUDA global memory of the current device, "host"
 *     pointers are ordinary host memory.  All device buffers are owned and
 *     allocated by the caller; the library never allocates device memory.
 *     pw_create allocates only a small host object.
 *   - Work is enqueued on the caller's stream and returns immediately.  Argument
 *     errors are detected on the host before anything is enqueued.  Problems met
 *     on the device (a bounded wait that ran out, a failed self check) are written
 *     to a status word that pw_last_device_status reads back.
 *   - Every device pointer must be 16-byte aligned.  rows and cols of a block
 *     must be multiples of 128.  Inputs must be finite.
 */
#ifndef PW_H_
#define PW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  PW_OK = 0,
  PW_ERR_INVALID_ARG = 1, /* null pointer, value out of range                         */
  PW_ERR_SHAPE = 2,       /* rows/cols not multiples of 128, shape differs from ctx   */
  PW_ERR_BITS = 3,        /* bitwidth not in {16,8,4,3,2}, or a demote that does not lower */
  PW_ERR_ALIGN = 4,       /* device pointer not 16-byte aligned                        */
  PW_ERR_STATE = 5,       /* page-table row missing, wrong page layout, not resident   */
  PW_ERR_NOMEM = 6,       /* caller's workspace too small                              */
  PW_ERR_CUDA = 7,        /* a CUDA runtime call failed                                */
  PW_ERR_TIMEOUT = 8      /* a bounded device-side wait ran out (see pw_last_device_status) */
} pw_status;

typedef enum { PW_GATE = 0, PW_UP = 1, PW_DOWN = 2 } pw_kind;

/* Which expert-FFN kernel family pw_moe_forward uses.  The paper's runtime has one kernel and no such switch
 * (Sec. 3.3); a caller leaves this at AUTO, which is TENSOR: the tensor-core kernels are the faster ones at
 * every batch size, one token included, and they pick the decode or the prefill instantiation (token tiles of
 * up to 64 or of 128) from the batch themselves.  SIMT is an independent second implementation kept for
 * cross-checks; it does not read PW_LAYOUT_PLANES pages. */
typedef enum {
  PW_MODE_AUTO = 0,
  PW_MODE_SIMT = 1,  /* CUDA-core kernel, thread per weight row: an independent second implementation */
  PW_MODE_TENSOR = 2 /* tcgen05 tensor-core kernel, pages dequantized into tensor memory      */
} pw_mode;

/* Page layouts.  CANONICAL: codes are a little-endian bit stream in row-major element
 * order (code of element n at stream bits [n*bits, (n+1)*bits)), scales / zero-points
 * fp16 [rows, cols/group] row-major; a 16-bit page is the fp16 matrix itself.
 * TILED: the same bytes regrouped per (128-row, one-group) tile so that a kernel reads a
 * tile with contiguous 16-byte loads; produced by pw_quantize_block / pw_demote_block /
 * pw_import_page and required by pw_moe_forward.  A TILED page is ONE buffer of the total
 * size pw_page_bytes returns, at `codes`: every tile is stored as its packed codes followed by
 * the 128 scales and the 128 zero-points of its rows, so a tile travels in a single copy;
 * `scales` and `zps` of a TILED page are ignored (may be NULL).  Both layouts have the same
 * total size. */
enum { PW_LAYOUT_CANONICAL = 0, PW_LAYOUT_TILED = 1, PW_LAYOUT_PLANES = 2 /* overlaid bit-planes, see below */ };

/* Residency state of a page-table row (Sec. 3.1).  Only GPU_RESIDENT rows can be used. */
enum {
  PW_STATE_GPU_RESIDENT = 0,
  PW_STATE_CPU_RESIDENT = 1,
  PW_STATE_IN_TRANSFER = 2,
  PW_STATE_NONE = 3 /* pw_page_state only: the library knows no page of the row at that bitwidth */
};

typedef struct CUstream_st* pw_stream; /* a cudaStream_t */
typedef struct pw_ctx pw_ctx;
typedef struct pw_page_table pw_page_table; /* the committed table of a context */

typedef struct {
  int32_t n_layers;   /* MoE layers the page table covers                        */
  int32_t n_experts;  /* routed experts E per layer                              */
  int32_t n_shared;   /* always-on shared experts per layer (gate 1, 16-bit pages) */
  int32_t hidden;     /* H, multiple of 128                                      */
  int32_t ffn;        /* F, expert FFN size, multiple of 128                     */
  int32_t group;      /* quantization group size; must be 128                    */
  int32_t max_tokens; /* largest T of a forward call                             */
  int32_t max_top_k;  /* largest top_k of a forward call                         */
  void* workspace;    /* device, >= pw_workspace_bytes(cfg), 256-byte aligned, owned by the caller,
                         must outlive the context; holds the committed table and all scratch   */
  size_t workspace_bytes;
} pw_config;

/* One weight page = one linear-block at one bitwidth (Sec. 3.1).  All pointers device. */
typedef struct {
  void* codes;    /* CANONICAL: packed codes, rows*cols*bits/8 bytes (bits == 16: fp16 weights);
                     TILED: the whole page, pw_page_bytes(...) bytes                             */
  void* scales;   /* CANONICAL, bits < 16: fp16, rows*cols/group values; otherwise ignored        */
  void* zps;      /* CANONICAL, bits < 16: fp16, rows*cols/group values; otherwise ignored        */
  uint32_t rows;  /* output features                                                            */
  uint32_t cols;  /* input features (the grouped, contracted dimension)                         */
  uint16_t group; /* 128                                                                        */
  uint8_t bits;   /* 16, 8, 4, 3 or 2 -- the committed bitwidth q_i once the row is published    */
  uint8_t layout; /* PW_LAYOUT_*                                                                */
} pw_page;

/* One page-table row, index i = (layer, expert, kind) (Sec. 3.1).  Experts
 * n_experts .. n_experts+n_shared-1 are the shared experts. */
typedef struct {
  int32_t layer, expert;
  int32_t kind;         /* pw_kind                                            */
  pw_page page;         /* page at the committed bitwidth q_i                 */
  uint8_t desired_bits; /* d_i chosen by a planner; recorded, not acted on    */
  uint8_t state;        /* PW_STATE_*; must be GPU_RESIDENT                   */
} pw_table_entry;

/* ---- context ------------------------------------------------------------------------ */

/* Bytes of device workspace a context with this configuration needs (0 if cfg is invalid). */
size_t pw_workspace_bytes(const pw_config* cfg);

/* Creates a context on the current device: the host object that holds the weight page table of Sec. 3.1 (one
 * row per (layer, expert, kind), at first empty) and the offsets of the routing and operand buffers of
 * Sec. 3.3 inside the caller's workspace.  cfg->workspace is zero-initialised and the call returns after that
 * has completed.
 * Errors: INVALID_ARG, SHAPE, ALIGN, NOMEM (workspace too small), CUDA. */
pw_status pw_create(pw_ctx** ctx, const pw_config* cfg);

/* Waits for the device, then frees the host object.  Device buffers stay with the caller. */
pw_status pw_destroy(pw_ctx* ctx);

/* Size table M_i^b of Eq. 3: total bytes of a rows x cols block at `bits`, metadata included;
 * the three parts are returned through the optional out pointers.  0 on invalid arguments.
 * Released bytes of a demotion b -> b' are pw_page_bytes(b) - pw_page_bytes(b'). */
size_t pw_page_bytes(uint32_t rows, uint32_t cols, int bits, int group, size_t* codes_bytes, size_t* scales_bytes,
                     size_t* zps_bytes);

/* ---- pages -------------------------------------------------------------------------- */

/* Group-quantizes an fp16 block into a new page.  w_fp16: device, [rows, cols] row-major.
 * dst: host struct whose `codes` points to a caller-allocated device buffer of the total size
 * pw_page_bytes reports (a TILED page is one buffer); the call fills rows, cols, group, bits,
 * layout (TILED).
 * bits == 16 stores the weights unchanged (a re-tiled copy).  Per group of 128 along cols, in
 * fp32 with one rounding per operation: lo = min, hi = max, scale = fp16((hi-lo)/(2^bits-1))
 * (1.0 if hi == lo, 2^-24 if it rounds to zero), zero-point = fp16(lo),
 * code = clamp(rint((w-lo) * (1/scale)), 0, 2^bits-1) with round-half-to-even.
 * The paper has no runtime quantizer (its lower precisions pre-exist as bit-plane subsets,
 * Sec. 2.2); this is the page constructor of this build's format.
 * Errors: INVALID_ARG, SHAPE, BITS, ALIGN. */
pw_status pw_quantize_block(pw_ctx* ctx, const void* w_fp16, uint32_t rows, uint32_t cols, int bits, pw_page* dst,
                            pw_stream stream);

/* Lowers a page: dst = quantize(dequantize(src), dst_bits), dst_bits < src->bits.  The offload
 * direction of Sec. 3.1 / 3.3: the new page is written to separate caller-allocated buffers, the
 * source is never modified, and the lower bitwidth takes effect only when the caller publishes
 * dst with pw_set_page_table.  src must be TILED.  Meant to run on a side stream while
 * pw_moe_forward runs on another.  Errors: INVALID_ARG, BITS, ALIGN, STATE (src not TILED). */
pw_status pw_demote_block(pw_ctx* ctx, const pw_page* src, int dst_bits, pw_page* dst, pw_stream stream);

/* Layout conversion, same bitwidth: TILED -> CANONICAL (export) and CANONICAL -> TILED (import).  What a page
 * row holds is Sec. 3.1's: the codes of the block at its committed bitwidth and the state needed to decode them
 * (here a scale and a zero-point per group); CANONICAL is that content in an order that does not depend on the
 * kernels.  dst buffers are caller-allocated, same sizes as src; the call fills dst's header fields.
 * Export is how pages are compared bit for bit and saved; import restores them.
 * Shapes (every page-building call): cols must be a multiple of the group size, 128, as the format asks, and
 * rows a multiple of 128 as well -- a TILED page is made of whole 128-row tiles (the MMA's M); the expert
 * matrices of the model families of Table 1 all satisfy both.  Anything else: PW_ERR_SHAPE.
 * Errors: INVALID_ARG, BITS, SHAPE, ALIGN, STATE (wrong source layout). */
pw_status pw_export_page(pw_ctx* ctx, const pw_page* src_tiled, pw_page* dst_canonical, pw_stream stream);
pw_status pw_import_page(pw_ctx* ctx, const pw_page* src_canonical, pw_page* dst_tiled, pw_stream stream);

/* ---- overlaid bit-plane pages --------------------------------------------------------- */

/* The paper's own page representation (Sec. 2.2 "Any-Precision"; Sec. 3.1: one bit-plane with its lookup-table
 * state is one weight page; Eq. 3: size table with the lookup-table metadata): a block is stored once as
 * overlaid bit-planes, a subset of the planes is a lower-precision version of the same block, and lowering the
 * precision computes nothing -- the planes above the committed bitwidth simply stop being read and may move to
 * host memory or be freed.  The paper does not say how its codes and centroids are fit; here the code is nested
 * on the group quantizer: master code c4 = the 4-bit code of pw_quantize_block, code at q bits = c4 >> (4 - q),
 * lookup table of q bits affine with scale_q = scale_4 * 2^(4-q) and zero-point_q = fp16(zero-point_4 +
 * scale_4 * (2^(4-q) - 1) / 2), the middle of the levels that the shorter code merges.  Supported q: 4, 3, 2.
 *
 * A PLANES block is three device buffers, carried by a pw_page with layout PW_LAYOUT_PLANES:
 *   codes  -> TOP   the two leading bits of every code, and the lookup-table state of all three bitwidths
 *   scales -> BIT1  the third bit   (needed for bits >= 3; may be NULL in a page published at 2 bits)
 *   zps    -> BIT0  the fourth bit  (needed for bits == 4; may be NULL below that)
 * and `bits` = the bitwidth it is read at.  pw_plane_bytes gives the buffer sizes (TOP, then each bit plane).
 * At q bits a forward call reads q/8 bytes per weight plus one lookup-table state per group: the bytes of
 * pw_page_bytes(rows, cols, q).
 *
 * pw_quantize_planes builds the three buffers from an fp16 block (device, [rows, cols] row-major) and fills the
 * header with bits = 4.  To lower or raise the precision the caller copies the header, sets `bits` (and may
 * clear the pointers of detached planes) and publishes it with pw_set_page_table: no kernel runs.
 * pw_export_planes writes the block's view at src->bits as a CANONICAL page (dst as for pw_export_page).
 * Errors: INVALID_ARG, SHAPE, BITS (bits outside 2..4), ALIGN, STATE (not a PLANES page; a needed plane is
 * detached). */
size_t pw_plane_bytes(uint32_t rows, uint32_t cols, size_t* top_bytes, size_t* bit_plane_bytes);
pw_status pw_quantize_planes(pw_ctx* ctx, const void* w_fp16, uint32_t rows, uint32_t cols, pw_page* dst,
                             pw_stream stream);
pw_status pw_export_planes(pw_ctx* ctx, const pw_page* src_planes, pw_page* dst_canonical, pw_stream stream);

/* ---- page table --------------------------------------------------------------------- */

/* Publishes n rows of the weight page table (Sec. 3.1): for each entry the row
 * (layer, expert, kind) now maps to entry.page with committed bitwidth page.bits.  Rows not
 * named keep their value (a row named twice takes its last entry).  The rows are carried to the device in
 * the parameters of a small kernel, so the update is ordered on `stream` like any kernel and does not wait
 * behind copies that other streams have queued on a DMA engine: forward calls enqueued on the same
 * stream before this call read the old rows, calls enqueued after it read the new rows -- the
 * "safe boundary" of Sec. 3.3 is the gap between two forward calls.  The previous page of a row
 * may be released once work enqueued before this call has finished.  entries: host.  epoch_out
 * (optional, host) receives the table epoch after the update; each call increments it by one.
 * Errors: INVALID_ARG, SHAPE (page shape does not match kind and ctx), BITS, ALIGN,
 * STATE (layout neither TILED nor PLANES, a plane the bitwidth needs is missing, state not GPU_RESIDENT, the page of the row at that bitwidth is CPU_RESIDENT or
 * IN_TRANSFER, shared expert below 16 bits), CUDA. */
pw_status pw_set_page_table(pw_ctx* ctx, const pw_table_entry* entries, size_t n, pw_stream stream,
                            uint64_t* epoch_out);

/* Handle of the committed table, for pw_moe_forward. */
const pw_page_table* pw_get_page_table(pw_ctx* ctx);

/* Host-side query of a committed row (what the last pw_set_page_table published). */
pw_status pw_query_row(pw_ctx* ctx, int layer, int expert, int kind, pw_table_entry* out);

/* ---- page residency: offload and reload ------------------------------------------------ */

/* The rest of a page's life-cycle (Sec. 3.1; Sec. 3.3, asynchronous page movement).  For every row and
 * every bitwidth the library keeps the residency state of the row's page at that bitwidth: a page
 * becomes GPU_RESIDENT when it is published with pw_set_page_table, and the calls below move it.  The
 * paper's two ordering rules are enforced on the host, before anything is enqueued:
 *   - offload: the committed bitwidth is lowered first, then the page that is no longer needed moves
 *     out -- the page a row is committed to cannot be offloaded (STATE);
 *   - reload: the page moves back first; pw_set_page_table refuses (STATE) a bitwidth whose page is
 *     CPU_RESIDENT or IN_TRANSFER, and accepts it once pw_page_state reports GPU_RESIDENT.
 * A TILED page is one buffer, so each direction is one asynchronous copy on `stream` (use a side stream
 * to overlap it with forward calls); host buffers should be pinned and are owned by the caller.
 *
 * pw_offload_page: copies `page` (device, TILED, pw_page_bytes bytes) of row (layer, expert, kind) to
 * host_dst; the page is IN_TRANSFER until the copy has finished, then CPU_RESIDENT.  The caller may
 * release the device buffer once pw_page_state reports CPU_RESIDENT and every forward call enqueued
 * before the commit that moved the row off this page has finished.
 * Errors: INVALID_ARG, SHAPE, BITS, ALIGN, STATE (not TILED; the row is committed to this page; the page
 * is already away or on its way), CUDA.
 *
 * pw_reload_page: copies the page of the row at `bits` from host_src (the buffer it was offloaded to)
 * into dst->codes (device, caller-allocated, pw_page_bytes bytes) and fills dst's header; IN_TRANSFER
 * until the copy has finished, then GPU_RESIDENT and ready for pw_set_page_table.
 * Errors: INVALID_ARG (also: host_src is not the buffer of the offload), SHAPE, BITS, ALIGN,
 * STATE (the page is not CPU_RESIDENT), CUDA.
 *
 * pw_page_state: the state now (looks at the transfer's event; never blocks); PW_STATE_NONE if the
 * library knows no page of the row at that bitwidth.
 *
 * pw_drop_page: forgets the page of the row at `bits` (its host copy is abandoned, or the caller is about
 * to build a new page at that bitwidth).  Errors: STATE (the row is committed to it; it is in transfer). */
pw_status pw_offload_page(pw_ctx* ctx, int layer, int expert, int kind, const pw_page* page, void* host_dst,
                          pw_stream stream);
pw_status pw_reload_page(pw_ctx* ctx, int layer, int expert, int kind, int bits, const void* host_src, pw_page* dst,
                         pw_stream stream);
pw_status pw_page_state(pw_ctx* ctx, int layer, int expert, int kind, int bits, int* state_out);
pw_status pw_drop_page(pw_ctx* ctx, int layer, int expert, int kind, int bits);

/* The same for a row that holds a block of overlaid bit-planes (PW_LAYOUT_PLANES), the paper's own case
 * (Sec. 2.2, Sec. 3.1): the unit of movement is a plane.  Plane 3 (the BIT1 buffer, at `scales` of the block's
 * header) is what reading at 3 bits adds to reading at 2 bits, plane 4 (BIT0, at `zps`) what 4 bits add to 3;
 * the leading planes (TOP) hold the table state of every bitwidth and never leave.  The two ordering rules,
 * checked on the host before anything is enqueued:
 *   - offload: a plane that the committed bitwidth of the row reads cannot leave (STATE) -- publish the block
 *     at a lower bitwidth first;
 *   - reload: pw_set_page_table refuses (STATE) a bitwidth that reads a plane which is CPU_RESIDENT or
 *     IN_TRANSFER, and accepts it once pw_plane_state reports GPU_RESIDENT (give the header the address the
 *     plane was reloaded to).
 * A plane is one buffer of `bit_bytes` (pw_plane_bytes), so each direction is one asynchronous copy on `stream`.
 * pw_offload_plane: block = the block's header (layout PLANES; only rows, cols and the plane's pointer are
 * used), plane = 3 or 4, host_dst = bit_bytes of (pinned) host memory.  The device buffer may be released once
 * pw_plane_state reports CPU_RESIDENT and every forward call enqueued before the commit that lowered the
 * bitwidth has finished.  Lowering the precision by q -> q' bits thus releases (q - q') * rows * cols / 8 bytes
 * of GPU memory (Eq. 3).
 * pw_reload_plane: host_src = the buffer the plane was offloaded to, dev_dst = bit_bytes of device memory.
 * Errors: INVALID_ARG (also: not the buffer of the offload), BITS (plane not 3 or 4), SHAPE, ALIGN, STATE, CUDA. */
pw_status pw_offload_plane(pw_ctx* ctx, int layer, int expert, int kind, const pw_page* block, int plane,
                           void* host_dst, pw_stream stream);
pw_status pw_reload_plane(pw_ctx* ctx, int layer, int expert, int kind, int plane, const void* host_src, void* dev_dst,
                          pw_stream stream);
pw_status pw_plane_state(pw_ctx* ctx, int layer, int expert, int kind, int plane, int* state_out);

/* ---- forward ------------------------------------------------------------------------ */

/* One MoE layer (Sec. 2.1, Sec. 3.3): top_k routing of T tokens over the E routed experts
 * (ties: lower expert index; gates = softmax over the k selected logits), stable grouping of
 * the (token, slot) pairs into per-expert segments, per expert y = W_down(silu(W_gate x) * W_up x)
 * with every block read at its committed bitwidth from `table`, and
 * out[t] = sum_j gate[t,j] * y_{e_j}[t] + sum over shared experts y_s[t].
 * hidden_fp16: device [T, H] fp16.  router_logits: device [T, E] fp32.  out: device [T, H] fp32.
 * table: pw_get_page_table(ctx) or NULL (same thing).  All rows of `layer` must have been
 * published.  Operands of the contractions are fp16, accumulation is fp32.
 * Errors: INVALID_ARG (T < 1, T > max_tokens, top_k < 1, top_k > min(E, max_top_k), bad layer),
 * ALIGN, STATE (a row of the layer is unpublished). */
pw_status pw_moe_forward(pw_ctx* ctx, int layer, const void* hidden_fp16, const float* router_logits, int T,
                         int top_k, const pw_page_table* table, float* out, pw_mode mode, pw_stream stream);

/* The same layer call for callers whose activations live in host memory: copies hidden_host
 * ([T, H] fp16) and logits_host ([T, E] fp32) to staging buffers in the workspace, runs
 * pw_moe_forward on them and copies the fp32 result to out_host ([T, H]), all ordered on `stream`.
 * The three host buffers should be pinned for the copies to be asynchronous, and must stay valid
 * until the stream has passed this call.  Calls that overlap on different streams would share the
 * staging buffers: use one stream per context.  Errors: as pw_moe_forward, plus CUDA. */
pw_status pw_moe_forward_host(pw_ctx* ctx, int layer, const void* hidden_host, const float* logits_host, int T,
                              int top_k, float* out_host, pw_mode mode, pw_stream stream);

/* The routing decision of the last forward call (Sec. 2.1: top-k experts per token and their gates; Sec. 3.3:
 * the grouping of the routed pairs by expert), copied out of the workspace (device pointers, any may
 * be NULL): topk_ids int32 [T, k], gates fp32 [T, k], counts int32 [E], offsets int32 [E+1],
 * perm int32 [T*k] (pair ids p = t*k + j sorted by expert, then by p). */
pw_status pw_get_routing(pw_ctx* ctx, int32_t* topk_ids, float* gates, int32_t* counts, int32_t* offsets,
                         int32_t* perm, pw_stream stream);

/* Routing for callers that cannot allocate device memory.  (The paper has no counterpart: this is
 * a convenience of this library.)  Some hosts of this code must not call cudaMalloc at all -- a
 * plug-in running inside another engine's memory pool, a process that has handed all device memory
 * to a caching allocator, code between the begin and end of a stream capture.  They cannot create a
 * context, because a context needs a workspace.  This call does the router and the stable grouping
 * of pw_moe_forward (same kernels, same results) and needs no context and no workspace: its scratch
 * (inverse permutation, row map, counters; about 0.5 MB) is a fixed array inside the library image,
 * which every GPU that has loaded the library holds until the process exits.
 *   router_logits: device [T, n_experts] fp32.  Outputs, all device and caller-allocated: topk_ids
 *   int32 [T, top_k], gates fp32 [T, top_k], counts int32 [n_experts], offsets int32 [n_experts + 1],
 *   perm int32 [T * top_k].
 * Limits: T * top_k <= 65536 and n_experts <= 256, else PW_ERR_NOMEM; top_k <= 32.
 * The first call on a device looks up the device address of the scratch array (one
 * cudaGetSymbolAddress with that device current); make that first call outside any stream capture.
 * The call allocates nothing, frees nothing and calls no allocating library routine.  All calls on a
 * device share the one scratch array: two calls that may run at the same time on the GPU (different
 * streams) race and must be ordered by the caller.  Calls on one stream are safe back to back; the
 * array keeps the previous call's contents and the kernels clear what they need to start from zero.
 * Errors: INVALID_ARG, ALIGN, NOMEM (over the limits), CUDA. */
pw_status pw_route_tokens_static(const float* router_logits, int T, int n_experts, int top_k, int32_t* topk_ids,
                                 float* gates, int32_t* counts, int32_t* offsets, int32_t* perm, pw_stream stream);

/* ---- observation taps ---------------------------------------------------------------- */

/* What a planner watches while the layer runs (Sec. 2.1, Sec. 3.2): the routing mass of every expert,
 * Eq. 1, and for every linear-block the three routed-input features -- routing-weighted mean input norm,
 * routing-weighted RMS input norm, maximum input norm -- of the tokens routed to the block's expert.
 * Both are ratios of sums over the observed (token, choice) pairs, so the library keeps the sums: per
 * layer and per expert segment s (routed experts, then shared experts) PW_OBS_FIELDS floats,
 *   SUM_R     sum of the routing weights r (the gates) of the pairs routed to s; a shared expert takes
 *             every token with r = 1
 *   PAIRS     number of those pairs
 *   SUM_R_NX, SUM_R_NX2, MAX_NX   sum r*|x|, sum r*|x|^2, max |x| with x the token's hidden state, the
 *             input of the gate and up blocks
 *   SUM_R_NH, SUM_R_NH2, MAX_NH   the same with h = silu(W_gate x) * (W_up x), the input of the down
 *             block, as the forward call computed it (fp16)
 * (the paper names the three features without a formula; |.| is the Euclidean norm).
 *
 * pw_observe(ctx, accumulators, stream): accumulators is a device array of
 * n_layers * (n_experts + n_shared) * PW_OBS_FIELDS floats owned by the caller; the call zeroes it on
 * `stream` and from then on every forward call of the context adds its tokens to the rows of its layer
 * (one small kernel at the end of the call, ordered on the call's stream; sums in a fixed order).
 * NULL switches the taps off.  The array must stay valid while the taps are on.
 * Errors: INVALID_ARG, ALIGN, CUDA. */
enum {
  PW_OBS_SUM_R = 0,
  PW_OBS_PAIRS = 1,
  PW_OBS_SUM_R_NX = 2,
  PW_OBS_SUM_R_NX2 = 3,
  PW_OBS_MAX_NX = 4,
  PW_OBS_SUM_R_NH = 5,
  PW_OBS_SUM_R_NH2 = 6,
  PW_OBS_MAX_NH = 7,
  PW_OBS_FIELDS = 8
};
pw_status pw_observe(pw_ctx* ctx, float* accumulators, pw_stream stream);

/* Turns the sums of one layer into the quantities themselves, on the device:
 *   mass (device, [n_experts] fp32, may be NULL): m_e = SUM_R[e] / sum over the routed experts (Eq. 1),
 *     zeros while nothing has been observed;
 *   phi (device, [(n_experts + n_shared) * 3 * 3] fp32, may be NULL): for segment s and kind u the triple
 *     (SUM_R_N / SUM_R, sqrt(SUM_R_N2 / SUM_R), MAX_N) at index (s * 3 + u) * 3, with the x sums for
 *     PW_GATE and PW_UP and the h sums for PW_DOWN; zeros for an expert without tokens.
 * Errors: INVALID_ARG, ALIGN, STATE (taps are off), CUDA. */
pw_status pw_observation_summary(pw_ctx* ctx, int layer, float* mass, float* phi, pw_stream stream);

/* ---- planner ------------------------------------------------------------------------- */

/* One scoring + selection step of the runtime planner (Sec. 3.2, Alg. 1).  Host code, no context and no GPU
 * needed; every pointer below is host memory.  A step lowers one linear-block from its current bitwidth to
 * the next lower bitwidth it supports; its predicted damage is
 *     d = max(epsilon, mu_bucket * g * eta)                                   (Eq. 8)
 *     g = max(s^{b'} - s^{b}, 0)                                              (Eq. 4)
 *     eta = exp(alpha * c * clip(w . phi + a, rho_min, rho_max))              (Eqs. 5-6; 1 without heads or
 *                                                                              for an expert that saw no token)
 * and the steps are taken cheapest damage per released byte first (ties: lower row index; a block's next step
 * becomes available when the one before has been taken) until `target` bytes are released.  The experts of a
 * layer are ranked by routing mass, hottest first, and bucket j holds the ranks below bucket_share[j] *
 * n_experts; a bucket has a damage multiplier and, per stage, a bitwidth floor.  Stages are tried in order:
 * the plan of the first stage that reaches the target is returned, otherwise the plan of the last stage (the
 * largest reduction the floors allow).  Shared experts are never touched.  The paper does not print its
 * calibrated constants (sensitivities, heads, buckets): they are the caller's.
 * Row index i = (layer * (n_experts + n_shared) + expert) * 3 + kind; bitwidth levels in the order 16, 8, 4, 3, 2. */
typedef struct {
  int32_t n_layers, n_experts, n_shared;
  const uint8_t* committed;     /* [rows] committed bitwidth q_i                                        */
  const uint8_t* supported;     /* [rows][5] non-zero where the block has a page at that level (B_i)    */
  const float* sensitivity;     /* [rows][5] offline sensitivity s_i^b                                  */
  const uint64_t* page_bytes;   /* [rows][5] size table M_i^b (Eq. 3), e.g. from pw_page_bytes          */
  const float* mass;            /* [n_layers][n_experts] routing mass (Eq. 1), e.g. pw_observation_summary */
  const float* phi;             /* [rows][3] routed-input features, or NULL                            */
  const float* head_w;          /* [3 kinds][5 from][5 to][3], or NULL: no prompt residual             */
  const float* head_a;          /* [3][5][5]                                                            */
  const float* head_c;          /* [3][5][5] confidence                                                 */
  float alpha, rho_min, rho_max, epsilon;
  int32_t n_buckets, n_stages;
  const float* bucket_share;    /* [n_buckets] ascending, the last one 1                                */
  const float* bucket_mu;       /* [n_buckets] damage multiplier, hottest bucket first                  */
  const uint8_t* stage_floor;   /* [n_stages][n_buckets] lowest bitwidth a bucket may reach in a stage  */
} pw_plan_tables;

typedef struct {
  int32_t layer, expert, kind;
  uint8_t from_bits, to_bits;
  uint64_t released_bytes;      /* M^{from} - M^{to}                                                    */
  double damage;                /* d of Eq. 8                                                           */
} pw_plan_item;

/* steps: array of max_steps items (may be NULL with max_steps 0 to ask for the count); n_steps_out
 * receives the number of steps of the plan, released_out (optional) their bytes, stage_out (optional) the
 * stage used.  Errors: INVALID_ARG, BITS (a committed bitwidth or floor outside the levels), NOMEM (the plan
 * has more than max_steps steps: nothing is written but the counts). */
pw_status pw_plan_step(const pw_plan_tables* tables, uint64_t target, pw_plan_item* steps, size_t max_steps,
                       size_t* n_steps_out, uint64_t* released_out, int32_t* stage_out);

/* The plan queue of Alg. 1.  The runtime calls the planner step again and again while requests run: every call
 * converts the KV-cache pressure into the byte target D_t (Eq. 7), builds one candidate plan per bitwidth-floor
 * stage (ScoreActions + GreedySelect) and keeps the candidates in the queue (RefreshPlanQueue), so that newer
 * observations replace older plans; only when the pressure is there (D_t > 0) does it hand out a plan
 * (SelectBestPlan: the candidate of the first stage that meets D_t, else the last stage's, the largest reduction
 * the floors allow).  Without pressure the candidates are prepared for `lookahead_bytes`, what the caller expects
 * to need next, and the call returns no steps (triggered_out = 0).  steps / max_steps / n_steps_out /
 * released_out / stage_out as for pw_plan_step.  pw_plan_queue_peek reports a stage's queued candidate (target
 * it was built for, bytes it releases, number of steps, the planner step that refreshed it).  Host code, no GPU.
 * Errors: INVALID_ARG (also: tables with another number of stages than the queue), BITS, NOMEM, STATE (peek of a
 * stage that has never been refreshed). */
typedef struct pw_plan_queue pw_plan_queue;
pw_status pw_plan_queue_create(pw_plan_queue** queue, int32_t n_stages);
pw_status pw_plan_queue_destroy(pw_plan_queue* queue);
pw_status pw_plan_queue_step(pw_plan_queue* queue, const pw_plan_tables* tables, int64_t free_block_threshold,
                             int64_t free_blocks, uint64_t kv_block_bytes, uint64_t lookahead_bytes, pw_plan_item* steps,
                             size_t max_steps, size_t* n_steps_out, uint64_t* released_out, int32_t* stage_out,
                             int32_t* triggered_out);
pw_status pw_plan_queue_peek(const pw_plan_queue* queue, int32_t stage, uint64_t* target_out, uint64_t* released_out,
                             size_t* n_steps_out, uint64_t* refreshed_at_out);

/* Eq. 7: bytes to release = max(0, free_block_threshold + 1 - free_blocks) * kv_block_bytes. */
uint64_t pw_kv_pressure_bytes(int64_t free_block_threshold, int64_t free_blocks, uint64_t kv_block_bytes);

/* ---- measurement and test aids (no counterpart in the paper) ----------------------------- */

/* Synchronises the device and returns the device status word (PW_OK, PW_ERR_TIMEOUT, ...),
 * then clears it. */
pw_status pw_last_device_status(pw_ctx* ctx);

/* Per-kernel device timing of pw_moe_forward (a measurement aid; off by default).  While enabled,
 * every forward call records CUDA events around each of its kernels on the caller's stream.
 * pw_kernel_timing(ctx, 1) enables and resets the sums, 0 disables.  pw_get_kernel_times waits for
 * the recorded events, adds up the elapsed milliseconds per kernel since the last reset into
 * ms_out[PW_NUM_KERNELS] (host) and returns the number of forward calls covered in calls_out (host).
 * The paper reports no per-kernel profile; this exists so that a benchmark can put a roofline
 * fraction on the dominant kernel. */
enum {
  PW_K_ROUTER = 0,
  PW_K_PERMUTE = 1,
  PW_K_GATHER = 2,
  PW_K_FFN_GATE_UP = 3,
  PW_K_FFN_DOWN = 4,
  PW_K_COMBINE = 5,
  PW_K_OBSERVE = 6, /* the kernel of the observation taps; ~0 while the taps are off */
  PW_NUM_KERNELS = 7
};
pw_status pw_kernel_timing(pw_ctx* ctx, int enable);
pw_status pw_get_kernel_times(pw_ctx* ctx, double* ms_out, uint64_t* calls_out);

/* Number of kernels the library has launched through this context since creation. */
uint64_t pw_launch_count(pw_ctx* ctx);

/* Test aid for the failure path of the expert-FFN kernels (the paper has no counterpart).  Every device-side
 * wait of those kernels is bounded, by 100000 polls of up to 20 us each (2 s).  The limit is compiled into the
 * kernels (carried in a register it cost the decode step 5 %), so `polls` only chooses: 0 = that default;
 * any other value = the gate/up kernel (narrow token tiles, ordinary pages) runs an instantiation whose limit
 * is 200 polls (4 ms).
 * When a wait runs out the CTA records PW_ERR_TIMEOUT in the status word, stops issuing work, frees its tensor
 * memory and returns; the call's output is then undefined and pw_last_device_status reports the timeout.
 * hook: 0 = none; bit 0 = the token-tile producer of the gate/up kernel stops before its second tile, so that
 * the waits on that tile run out -- the one safe way to exercise the path (nothing faults, traps or spins
 * without a limit).  Applies to forward calls enqueued after it.  Errors: INVALID_ARG. */
pw_status pw_debug_set_wait(pw_ctx* ctx, uint32_t polls, uint32_t hook);

const char* pw_status_str(pw_status s);

#ifdef __cplusplus
}
#endif
#endif /* PW_H_ */
