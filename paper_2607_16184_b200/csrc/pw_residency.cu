// Page life-cycle beyond the GPU: residency records, offload to host memory and reload (Sec. 3.1, Sec. 3.3
// "asynchronous page movement").  A page leaves only after the committed bitwidth of its row has moved off
// it, and a bitwidth is committed only while its page is GPU-resident; both rules are checked on the host
// before anything is enqueued.  The bytes travel with one asynchronous copy per page on the caller's stream
// (a TILED page is a single buffer), so a side stream overlaps them with forward calls on another.
#include "pw_common.cuh"

namespace pw {

static PageRecord* record_of(pw_ctx* ctx, size_t row, int bits) {
  const int lv = bit_level(bits);
  return lv < 0 ? nullptr : &ctx->records[row * kBitLevels + lv];
}

// A transfer whose event has completed has arrived.
int residency_poll(pw_ctx* ctx, size_t row, int bits) {
  PageRecord* r = record_of(ctx, row, bits);
  if (!r) return PW_STATE_NONE;
  if (r->state == PW_STATE_IN_TRANSFER && r->ev && cudaEventQuery(r->ev) == cudaSuccess) {
    r->state = r->heading;
    if (r->state == PW_STATE_CPU_RESIDENT) r->dev = nullptr;
  }
  return r->state;
}

pw_status residency_check_commit(pw_ctx* ctx, size_t row, const pw_page& page) {
  const int st = residency_poll(ctx, row, page.bits);
  if (st == PW_STATE_IN_TRANSFER || st == PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  return PW_OK;
}

void residency_note_commit(pw_ctx* ctx, size_t row, const pw_page& page) {
  PageRecord* r = record_of(ctx, row, page.bits);
  if (!r) return;
  r->state = PW_STATE_GPU_RESIDENT;
  r->dev = page.codes;
}

static int poll_record(PageRecord* r) {
  if (r->state == PW_STATE_IN_TRANSFER && r->ev && cudaEventQuery(r->ev) == cudaSuccess) {
    r->state = r->heading;
    if (r->state == PW_STATE_CPU_RESIDENT) r->dev = nullptr;
  }
  return r->state;
}

// A block of bit-planes read at q bits needs the planes 3 .. q on the GPU (Sec. 3.1: the bitwidth is raised only
// once the planes it reads are back).
pw_status residency_check_commit_planes(pw_ctx* ctx, size_t row, const pw_page& page) {
  for (int p = 3; p <= page.bits; ++p) {
    const int st = poll_record(&ctx->records[row * kBitLevels + plane_level(p)]);
    if (st == PW_STATE_IN_TRANSFER || st == PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  }
  return PW_OK;
}

void residency_note_commit_planes(pw_ctx* ctx, size_t row, const pw_page& page) {
  for (int p = 3; p <= page.bits; ++p) {
    PageRecord* r = &ctx->records[row * kBitLevels + plane_level(p)];
    r->state = PW_STATE_GPU_RESIDENT;
    r->dev = p == 3 ? page.scales : page.zps;
  }
}

void residency_teardown(pw_ctx* ctx) {
  if (!ctx->records) return;
  for (size_t i = 0; i < ctx->n_rows * kBitLevels; ++i)
    if (ctx->records[i].ev) cudaEventDestroy(ctx->records[i].ev);
  delete[] ctx->records;
  ctx->records = nullptr;
}

static pw_status check_row_page(const pw_ctx* ctx, int layer, int expert, int kind, uint32_t rows, uint32_t cols,
                                int bits) {
  const pw_config& c = ctx->cfg;
  if (layer < 0 || layer >= c.n_layers || expert < 0 || expert >= ctx->ws.S || kind < 0 || kind > 2)
    return PW_ERR_INVALID_ARG;
  if (bit_level(bits) < 0) return PW_ERR_BITS;
  const uint32_t er = kind == PW_DOWN ? c.hidden : c.ffn, ec = kind == PW_DOWN ? c.ffn : c.hidden;
  if (rows != er || cols != ec) return PW_ERR_SHAPE;
  return PW_OK;
}

static pw_status start_transfer(PageRecord* r, void* dst, const void* src, size_t bytes, cudaMemcpyKind dir,
                                cudaStream_t stream) {
  if (!r->ev) PW_CUDA_OK(cudaEventCreateWithFlags(&r->ev, cudaEventDisableTiming));
  PW_CUDA_OK(cudaMemcpyAsync(dst, src, bytes, dir, stream));
  PW_CUDA_OK(cudaEventRecord(r->ev, stream));
  return PW_OK;
}

}  // namespace pw

using namespace pw;

extern "C" pw_status pw_offload_page(pw_ctx* ctx, int layer, int expert, int kind, const pw_page* page, void* host_dst,
                                     pw_stream stream) {
  if (!ctx || !page || !host_dst || !page->codes) return PW_ERR_INVALID_ARG;
  pw_status st = check_row_page(ctx, layer, expert, kind, page->rows, page->cols, page->bits);
  if (st != PW_OK) return st;
  if (page->layout != PW_LAYOUT_TILED || page->group != kGroup) return PW_ERR_STATE;
  if (reinterpret_cast<uintptr_t>(page->codes) & 15) return PW_ERR_ALIGN;
  const size_t row = row_index(ctx, layer, expert, kind);
  // the committed bitwidth is lowered first, then the page that is no longer needed moves out
  if (ctx->host_valid[row] && ctx->host_rows[row].page.bits == page->bits) return PW_ERR_STATE;
  const int cur = residency_poll(ctx, row, page->bits);
  if (cur == PW_STATE_IN_TRANSFER || cur == PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  PageRecord* r = &ctx->records[row * kBitLevels + bit_level(page->bits)];
  const size_t bytes = pw_page_bytes(page->rows, page->cols, page->bits, kGroup, nullptr, nullptr, nullptr);
  st = start_transfer(r, host_dst, page->codes, bytes, cudaMemcpyDeviceToHost, stream);
  if (st != PW_OK) return st;
  r->state = PW_STATE_IN_TRANSFER;
  r->heading = PW_STATE_CPU_RESIDENT;
  r->dev = page->codes;
  r->host = host_dst;
  return PW_OK;
}

extern "C" pw_status pw_reload_page(pw_ctx* ctx, int layer, int expert, int kind, int bits, const void* host_src,
                                    pw_page* dst, pw_stream stream) {
  if (!ctx || !host_src || !dst || !dst->codes) return PW_ERR_INVALID_ARG;
  const pw_config& c = ctx->cfg;
  const uint32_t rows = kind == PW_DOWN ? c.hidden : c.ffn, cols = kind == PW_DOWN ? c.ffn : c.hidden;
  pw_status st = check_row_page(ctx, layer, expert, kind, rows, cols, bits);
  if (st != PW_OK) return st;
  if (reinterpret_cast<uintptr_t>(dst->codes) & 15) return PW_ERR_ALIGN;
  const size_t row = row_index(ctx, layer, expert, kind);
  if (residency_poll(ctx, row, bits) != PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  PageRecord* r = &ctx->records[row * kBitLevels + bit_level(bits)];
  if (r->host != host_src) return PW_ERR_INVALID_ARG;     // not the buffer this page was offloaded to
  const size_t bytes = pw_page_bytes(rows, cols, bits, kGroup, nullptr, nullptr, nullptr);
  st = start_transfer(r, dst->codes, host_src, bytes, cudaMemcpyHostToDevice, stream);
  if (st != PW_OK) return st;
  r->state = PW_STATE_IN_TRANSFER;
  r->heading = PW_STATE_GPU_RESIDENT;
  r->dev = dst->codes;
  dst->rows = rows;
  dst->cols = cols;
  dst->group = kGroup;
  dst->bits = (uint8_t)bits;
  dst->layout = PW_LAYOUT_TILED;
  return PW_OK;
}

extern "C" pw_status pw_drop_page(pw_ctx* ctx, int layer, int expert, int kind, int bits) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers || expert < 0 || expert >= ctx->ws.S || kind < 0 || kind > 2)
    return PW_ERR_INVALID_ARG;
  if (bit_level(bits) < 0) return PW_ERR_BITS;
  const size_t row = row_index(ctx, layer, expert, kind);
  if (ctx->host_valid[row] && ctx->host_rows[row].page.bits == bits) return PW_ERR_STATE;   // the committed page
  if (residency_poll(ctx, row, bits) == PW_STATE_IN_TRANSFER) return PW_ERR_STATE;           // let it arrive first
  PageRecord* r = &ctx->records[row * kBitLevels + bit_level(bits)];
  r->state = PW_STATE_NONE;
  r->dev = r->host = nullptr;
  return PW_OK;
}

extern "C" pw_status pw_page_state(pw_ctx* ctx, int layer, int expert, int kind, int bits, int* state_out) {
  if (!ctx || !state_out) return PW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers || expert < 0 || expert >= ctx->ws.S || kind < 0 || kind > 2)
    return PW_ERR_INVALID_ARG;
  if (bit_level(bits) < 0) return PW_ERR_BITS;
  *state_out = residency_poll(ctx, row_index(ctx, layer, expert, kind), bits);
  return PW_OK;
}

// ---- planes of a bit-plane block ---------------------------------------------------------------

static pw_status check_plane_args(const pw_ctx* ctx, int layer, int expert, int kind, int plane) {
  if (layer < 0 || layer >= ctx->cfg.n_layers || expert < 0 || expert >= ctx->ws.S || kind < 0 || kind > 2)
    return PW_ERR_INVALID_ARG;
  return plane_level(plane) < 0 ? PW_ERR_BITS : PW_OK;
}

extern "C" pw_status pw_offload_plane(pw_ctx* ctx, int layer, int expert, int kind, const pw_page* block, int plane,
                                      void* host_dst, pw_stream stream) {
  if (!ctx || !block || !host_dst) return PW_ERR_INVALID_ARG;
  pw_status st = check_plane_args(ctx, layer, expert, kind, plane);
  if (st != PW_OK) return st;
  if (block->layout != PW_LAYOUT_PLANES || block->group != kGroup) return PW_ERR_STATE;
  const pw_config& c = ctx->cfg;
  const uint32_t er = kind == PW_DOWN ? c.hidden : c.ffn, ec = kind == PW_DOWN ? c.ffn : c.hidden;
  if (block->rows != er || block->cols != ec) return PW_ERR_SHAPE;
  void* dev = plane == 3 ? block->scales : block->zps;
  if (!dev) return PW_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dev) & 15) return PW_ERR_ALIGN;
  const size_t row = row_index(ctx, layer, expert, kind);
  // the committed bitwidth is lowered first, then the plane it no longer reads moves out
  const pw_page& cur = ctx->host_rows[row].page;
  if (ctx->host_valid[row] && cur.layout == PW_LAYOUT_PLANES && cur.bits >= plane) return PW_ERR_STATE;
  PageRecord* r = &ctx->records[row * kBitLevels + plane_level(plane)];
  const int now = poll_record(r);
  if (now == PW_STATE_IN_TRANSFER || now == PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  size_t bit_bytes = 0;
  pw_plane_bytes(block->rows, block->cols, nullptr, &bit_bytes);
  st = start_transfer(r, host_dst, dev, bit_bytes, cudaMemcpyDeviceToHost, stream);
  if (st != PW_OK) return st;
  r->state = PW_STATE_IN_TRANSFER;
  r->heading = PW_STATE_CPU_RESIDENT;
  r->dev = dev;
  r->host = host_dst;
  return PW_OK;
}

extern "C" pw_status pw_reload_plane(pw_ctx* ctx, int layer, int expert, int kind, int plane, const void* host_src,
                                     void* dev_dst, pw_stream stream) {
  if (!ctx || !host_src || !dev_dst) return PW_ERR_INVALID_ARG;
  pw_status st = check_plane_args(ctx, layer, expert, kind, plane);
  if (st != PW_OK) return st;
  if (reinterpret_cast<uintptr_t>(dev_dst) & 15) return PW_ERR_ALIGN;
  const size_t row = row_index(ctx, layer, expert, kind);
  PageRecord* r = &ctx->records[row * kBitLevels + plane_level(plane)];
  if (poll_record(r) != PW_STATE_CPU_RESIDENT) return PW_ERR_STATE;
  if (r->host != host_src) return PW_ERR_INVALID_ARG;     // not the buffer this plane was offloaded to
  const pw_config& c = ctx->cfg;
  size_t bit_bytes = 0;
  pw_plane_bytes(kind == PW_DOWN ? c.hidden : c.ffn, kind == PW_DOWN ? c.ffn : c.hidden, nullptr, &bit_bytes);
  st = start_transfer(r, dev_dst, host_src, bit_bytes, cudaMemcpyHostToDevice, stream);
  if (st != PW_OK) return st;
  r->state = PW_STATE_IN_TRANSFER;
  r->heading = PW_STATE_GPU_RESIDENT;
  r->dev = dev_dst;
  return PW_OK;
}

extern "C" pw_status pw_plane_state(pw_ctx* ctx, int layer, int expert, int kind, int plane, int* state_out) {
  if (!ctx || !state_out) return PW_ERR_INVALID_ARG;
  const pw_status st = check_plane_args(ctx, layer, expert, kind, plane);
  if (st != PW_OK) return st;
  PageRecord* r = &ctx->records[row_index(ctx, layer, expert, kind) * kBitLevels + plane_level(plane)];
  *state_out = poll_record(r);
  return PW_OK;
}
