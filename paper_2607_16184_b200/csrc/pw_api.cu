// Context, workspace map, page-table commits and the forward-call orchestration.
#include <new>
#include <string.h>

#include "pw_common.cuh"

namespace pw {

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
static bool bits_ok(int b) { return b == 16 || b == 8 || b == 4 || b == 3 || b == 2; }

static bool config_ok(const pw_config& c) {
  if (c.n_layers < 1 || c.n_experts < 1 || c.n_experts > 256 || c.n_shared < 0 || c.n_shared > 16) return false;
  if (c.hidden < kGroup || c.ffn < kGroup || c.hidden % kGroup || c.ffn % kGroup) return false;
  if (c.group != kGroup) return false;
  if (c.max_tokens < 1 || c.max_top_k < 1 || c.max_top_k > 32 || c.max_top_k > c.n_experts) return false;
  if ((long long)c.max_tokens * (c.max_top_k + c.n_shared) > (1ll << 24)) return false;
  return true;
}

WsMap make_wsmap(const pw_config& c) {
  WsMap m{};
  m.S = c.n_experts + c.n_shared;
  const int P = c.max_tokens * c.max_top_k;
  m.Rmax = P + c.n_shared * c.max_tokens;
  m.Rpad = m.Rmax + kPadRows;
  const int maxdim = c.hidden > c.ffn ? c.hidden : c.ffn;
  m.max_units = (m.Rmax / 16 + m.S + 1) * (maxdim / kTileRows) * 8;
  const size_t eight = (size_t)8 * m.Rmax;
  m.y_slots = eight < 8192 ? eight : ((size_t)m.Rmax > 8192 ? (size_t)m.Rmax : 8192);
  size_t o = 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o = align_up(o + bytes, 256);
    return at;
  };
  m.status = take(64 * 4);
  m.counter = take(64 * 4);
  m.table = take(sizeof(DevRow) * (size_t)c.n_layers * m.S * 3);
  m.topk_ids = take(4 * (size_t)P);
  m.gates = take(4 * (size_t)P);
  m.counts = take(4 * (size_t)m.S);
  m.offsets = take(4 * (size_t)(m.S + 1));
  m.perm = take(4 * (size_t)P);
  m.inv_perm = take(4 * (size_t)P);
  m.row_token = take(4 * (size_t)m.Rpad);
  m.seg_order = take(4 * (size_t)m.S);
  m.max_tiles = m.Rmax / 16 + m.S + 8;
  m.tile_tab = take(2 * 8 * (size_t)m.max_tiles);
  m.units_gu = take(sizeof(Unit) * (size_t)m.max_units);
  m.units_dn = take(sizeof(Unit) * (size_t)m.max_units);
  m.n_units = take(16);
  m.done = take(4 * 8 * (size_t)m.Rmax);
  m.xt = take((size_t)c.hidden * 2 * m.Rpad);
  m.ht = take((size_t)c.ffn * 2 * m.Rpad);
  m.y = take(m.y_slots * c.hidden * 4);
  m.io_hidden = take((size_t)c.max_tokens * c.hidden * 2);
  m.io_logits = take((size_t)c.max_tokens * c.n_experts * 4);
  m.io_out = take((size_t)c.max_tokens * c.hidden * 4);
  m.obs_part = take(4 * (size_t)kNormSplit * 2 * m.Rpad);
  m.total = o;
  return m;
}

// Rows of one page-table update, passed by value to the kernel that writes them (3.3 KB of the 4 KB a kernel's
// parameters may take).
constexpr int kCommitBatch = 64;
struct CommitBatch {
  int n;
  uint32_t index[kCommitBatch];
  DevRow row[kCommitBatch];
};
__global__ void __launch_bounds__(kCommitBatch) commit_rows_kernel(const __grid_constant__ CommitBatch batch,
                                                                  DevRow* __restrict__ table) {
  const int j = threadIdx.x;
  if (j < batch.n) table[batch.index[j]] = batch.row[j];
}

static void timing_drain_slot(pw_ctx* ctx, int slot) {
  if (!ctx->timing_busy[slot]) return;
  cudaEvent_t* ev = ctx->timing_ev + (size_t)slot * (PW_NUM_KERNELS + 1);
  if (cudaEventSynchronize(ev[PW_NUM_KERNELS]) == cudaSuccess) {
    for (int i = 0; i < PW_NUM_KERNELS; ++i) {
      float ms = 0.f;
      if (cudaEventElapsedTime(&ms, ev[i], ev[i + 1]) == cudaSuccess) ctx->timing_ms[i] += ms;
    }
    ctx->timing_calls++;
  }
  ctx->timing_busy[slot] = false;
}

void timing_mark(pw_ctx* ctx, int i, cudaStream_t s) {
  if (!ctx->timing_on) return;
  cudaEventRecord(ctx->timing_ev[(size_t)ctx->timing_cur * (PW_NUM_KERNELS + 1) + i], s);
}

}  // namespace pw

using namespace pw;

extern "C" size_t pw_workspace_bytes(const pw_config* cfg) {
  if (!cfg || !config_ok(*cfg)) return 0;
  return make_wsmap(*cfg).total;
}

extern "C" pw_status pw_create(pw_ctx** out, const pw_config* cfg) {
  if (!out || !cfg) return PW_ERR_INVALID_ARG;
  *out = nullptr;
  if (cfg->group != kGroup || cfg->hidden % kGroup || cfg->ffn % kGroup) return PW_ERR_SHAPE;
  if (!config_ok(*cfg) || !cfg->workspace) return PW_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cfg->workspace) & 255) return PW_ERR_ALIGN;
  WsMap m = make_wsmap(*cfg);
  if (cfg->workspace_bytes < m.total) return PW_ERR_NOMEM;
  pw_ctx* ctx = new (std::nothrow) pw_ctx();
  if (!ctx) return PW_ERR_NOMEM;
  ctx->cfg = *cfg;
  ctx->ws = m;
  ctx->base = reinterpret_cast<char*>(cfg->workspace);
  ctx->table_handle.owner = ctx;
  ctx->epoch = 0;
  ctx->launches = 0;
  ctx->last_T = ctx->last_k = 0;
  ctx->tc_state = nullptr;
  ctx->wait_polls = 0;
  ctx->test_hook = 0;
  ctx->timing_on = false;
  ctx->timing_ev = nullptr;
  ctx->timing_cur = 0;
  ctx->timing_calls = 0;
  ctx->obs_acc = nullptr;
  for (int i = 0; i < pw_ctx::kTimingSlots; ++i) ctx->timing_busy[i] = false;
  for (int i = 0; i < PW_NUM_KERNELS; ++i) ctx->timing_ms[i] = 0.0;
  const size_t nrows = (size_t)cfg->n_layers * m.S * 3;
  ctx->n_rows = nrows;
  ctx->host_rows = new (std::nothrow) pw_table_entry[nrows]();
  ctx->host_valid = new (std::nothrow) uint8_t[nrows]();
  ctx->records = new (std::nothrow) PageRecord[nrows * kBitLevels]();
  for (size_t i = 0; ctx->records && i < nrows * kBitLevels; ++i) ctx->records[i].state = PW_STATE_NONE;
  bool ok = ctx->host_rows && ctx->host_valid && ctx->records;
  int dev = 0;
  ok = ok && cudaGetDevice(&dev) == cudaSuccess;
  ok = ok && cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess;
  // the table (valid = 0), status word, counters and operand padding start out as zeros
  ok = ok && cudaMemset(ctx->base, 0, m.total) == cudaSuccess;
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    pw_destroy(ctx);
    return PW_ERR_CUDA;
  }
  *out = ctx;
  return PW_OK;
}

extern "C" pw_status pw_destroy(pw_ctx* ctx) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  tc_teardown(ctx);
  if (ctx->timing_ev) {
    for (int i = 0; i < pw_ctx::kTimingSlots * (PW_NUM_KERNELS + 1); ++i)
      if (ctx->timing_ev[i]) cudaEventDestroy(ctx->timing_ev[i]);
    delete[] ctx->timing_ev;
  }
  residency_teardown(ctx);
  delete[] ctx->host_rows;
  delete[] ctx->host_valid;
  delete ctx;
  return PW_OK;
}

extern "C" pw_status pw_set_page_table(pw_ctx* ctx, const pw_table_entry* entries, size_t n, pw_stream stream,
                                       uint64_t* epoch_out) {
  if (!ctx || (!entries && n)) return PW_ERR_INVALID_ARG;
  const pw_config& c = ctx->cfg;
  if (n > ctx->n_rows) return PW_ERR_INVALID_ARG;
  // validate everything before anything is enqueued
  for (size_t i = 0; i < n; ++i) {
    const pw_table_entry& e = entries[i];
    const pw_page& p = e.page;
    if (e.layer < 0 || e.layer >= c.n_layers || e.expert < 0 || e.expert >= ctx->ws.S || e.kind < 0 || e.kind > 2)
      return PW_ERR_INVALID_ARG;
    const bool planes = p.layout == PW_LAYOUT_PLANES;
    if (planes ? (p.bits < 2 || p.bits > 4) : !bits_ok(p.bits)) return PW_ERR_BITS;
    const uint32_t er = e.kind == PW_DOWN ? c.hidden : c.ffn, ec = e.kind == PW_DOWN ? c.ffn : c.hidden;
    if (p.rows != er || p.cols != ec || p.group != kGroup) return PW_ERR_SHAPE;
    if (!p.codes) return PW_ERR_INVALID_ARG;   // a TILED page is one buffer: scales and zero-points sit inside it
    if (!aligned16(p.codes)) return PW_ERR_ALIGN;
    if ((p.layout != PW_LAYOUT_TILED && !planes) || e.state != PW_STATE_GPU_RESIDENT) return PW_ERR_STATE;
    if (planes) {
      // the bitwidth is only set to what the attached planes can give (Sec. 3.1)
      if ((p.bits >= 3 && !p.scales) || (p.bits == 4 && !p.zps)) return PW_ERR_STATE;
      if (!aligned16(p.scales) || !aligned16(p.zps)) return PW_ERR_ALIGN;
    }
    if (e.expert >= c.n_experts && (p.bits != 16 || planes)) return PW_ERR_STATE;
    if (e.desired_bits != 0 && !bits_ok(e.desired_bits)) return PW_ERR_BITS;
    // q_i is only set to a bitwidth whose page is GPU-resident (Sec. 3.1): not while it is away or on its way
    const size_t ridx = row_index(ctx, e.layer, e.expert, e.kind);
    const pw_status rs = planes ? residency_check_commit_planes(ctx, ridx, p) : residency_check_commit(ctx, ridx, p);
    if (rs != PW_OK) return rs;
  }
  // The rows travel in the parameter space of a small kernel, 64 at a time: the update is ordered on the
  // stream like any kernel and never queues behind a large copy on a DMA engine (a page being reloaded on a
  // side stream would otherwise hold up the commits of the stream that runs the forward calls).
  DevRow* dtab = reinterpret_cast<DevRow*>(ctx->base + ctx->ws.table);
  size_t i = 0;
  while (i < n) {
    CommitBatch batch;
    batch.n = 0;
    for (; i < n && batch.n < kCommitBatch; ++i) {
      const pw_table_entry& e = entries[i];
      DevRow r{};
      r.codes = e.page.codes;
      r.rows = e.page.rows;
      r.cols = e.page.cols;
      r.bits = e.page.bits;
      r.valid = e.page.layout == PW_LAYOUT_PLANES ? 2 : 1;
      r.bit1 = r.valid == 2 ? e.page.scales : nullptr;
      r.bit0 = r.valid == 2 ? e.page.zps : nullptr;
      const size_t idx = row_index(ctx, e.layer, e.expert, e.kind);
      int j = 0;                                   // a row named twice keeps its last entry
      while (j < batch.n && batch.index[j] != (uint32_t)idx) ++j;
      batch.row[j] = r;
      batch.index[j] = (uint32_t)idx;
      if (j == batch.n) ++batch.n;
      ctx->host_rows[idx] = e;
      ctx->host_valid[idx] = 1;
      if (e.page.layout != PW_LAYOUT_PLANES) residency_note_commit(ctx, idx, e.page);
      else residency_note_commit_planes(ctx, idx, e.page);
    }
    commit_rows_kernel<<<1, kCommitBatch, 0, stream>>>(batch, dtab);
    ctx->launches++;
    PW_CUDA_OK(cudaGetLastError());
  }
  ctx->epoch++;
  if (epoch_out) *epoch_out = ctx->epoch;
  return PW_OK;
}

extern "C" const pw_page_table* pw_get_page_table(pw_ctx* ctx) { return ctx ? &ctx->table_handle : nullptr; }

extern "C" pw_status pw_query_row(pw_ctx* ctx, int layer, int expert, int kind, pw_table_entry* out) {
  if (!ctx || !out) return PW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers || expert < 0 || expert >= ctx->ws.S || kind < 0 || kind > 2)
    return PW_ERR_INVALID_ARG;
  const size_t idx = row_index(ctx, layer, expert, kind);
  if (!ctx->host_valid[idx]) return PW_ERR_STATE;
  *out = ctx->host_rows[idx];
  return PW_OK;
}

// Argument checks of a forward call: everything that can be refused is refused here, before anything is enqueued.
static pw_status check_forward_args(pw_ctx* ctx, int layer, const void* hidden, const float* logits, int T, int top_k,
                                    const pw_page_table* table, const float* out, pw_mode mode) {
  if (!ctx || !hidden || !logits || !out) return PW_ERR_INVALID_ARG;
  const pw_config& c = ctx->cfg;
  if (table && table->owner != ctx) return PW_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c.n_layers || T < 1 || T > c.max_tokens || top_k < 1 || top_k > c.max_top_k ||
      top_k > c.n_experts)
    return PW_ERR_INVALID_ARG;
  if (mode != PW_MODE_AUTO && mode != PW_MODE_SIMT && mode != PW_MODE_TENSOR) return PW_ERR_INVALID_ARG;
  if (!aligned16(hidden) || !aligned16(logits) || !aligned16(out)) return PW_ERR_ALIGN;
  for (int e = 0; e < ctx->ws.S; ++e)
    for (int u = 0; u < 3; ++u)
      if (!ctx->host_valid[row_index(ctx, layer, e, u)]) return PW_ERR_STATE;
  if (mode == PW_MODE_SIMT)                      // the CUDA-core kernel reads TILED pages only
    for (int e = 0; e < ctx->ws.S; ++e)
      for (int u = 0; u < 3; ++u)
        if (ctx->host_rows[row_index(ctx, layer, e, u)].page.layout == PW_LAYOUT_PLANES) return PW_ERR_STATE;
  return PW_OK;
}

extern "C" pw_status pw_moe_forward(pw_ctx* ctx, int layer, const void* hidden, const float* logits, int T, int top_k,
                                    const pw_page_table* table, float* out, pw_mode mode, pw_stream stream) {
  const pw_status as = check_forward_args(ctx, layer, hidden, logits, T, top_k, table, out, mode);
  if (as != PW_OK) return as;
  const pw_config& c = ctx->cfg;

  // The tensor-core kernels win at every batch size measured (one token of a Mixtral-shaped layer: 0.12 ms
  // against 1.96 ms for the CUDA-core kernel), so AUTO means TENSOR; the CUDA-core kernel stays selectable as
  // an independent second implementation.
  if (mode == PW_MODE_AUTO) mode = PW_MODE_TENSOR;
  int nt_tile = 0, ksplit = 1;
  if (mode == PW_MODE_TENSOR) {
    nt_tile = tensor_token_tile(ctx, T, top_k);
    // split the down projection's contraction until there are a few units per SM
    const int R = T * top_k + c.n_shared * T;
    const int active = ctx->ws.S < R ? ctx->ws.S : R;
    const long long tiles = (long long)active * ((R / active + nt_tile - 1) / nt_tile) * (c.hidden / kTileRows);
    // Pick the split (1..8) that finishes soonest under a simple cost model: the CTAs (one per SM) work through
    // ceil(units / SMs) rounds of units, and a unit costs a fixed part -- claiming it, the accumulator
    // hand-over, the epilogue: about three tiles' worth of time, measured -- plus one part per 128-wide tile of
    // its K range.  A finer split fills the last round better but multiplies the fixed parts, so it only pays
    // when units are long (an 8-expert layer with F = 14336: split 4); layers with short contractions or many
    // small experts are fastest unsplit.  On ties the smaller split (less partial traffic).
    const int ng = c.ffn / kGroup;
    const long long G = ctx->num_sms;
    long long want = 1, best = -1;
    for (int ks = 1; ks <= 8 && ks <= ng; ++ks) {
      if ((size_t)ks * R > ctx->ws.y_slots) break;
      const long long rounds = (tiles * ks + G - 1) / G;
      const long long cost = rounds * (3 + (ng + ks - 1) / ks);
      if (best < 0 || cost < best) {
        best = cost;
        want = ks;
      }
    }
    ksplit = (int)want;
  }
  if (ctx->timing_on) {
    ctx->timing_cur = (ctx->timing_cur + 1) % pw_ctx::kTimingSlots;
    timing_drain_slot(ctx, ctx->timing_cur);   // waits only when the ring has wrapped onto unfinished work
    ctx->timing_busy[ctx->timing_cur] = true;
  }
  pw_status st = launch_route(ctx, layer, hidden, logits, T, top_k, nt_tile, ksplit, stream);
  if (st != PW_OK) return st;
  st = mode == PW_MODE_SIMT ? launch_ffn_simt(ctx, layer, T, top_k, stream)
                            : launch_ffn_tensor(ctx, layer, T, top_k, nt_tile, ksplit, stream);
  if (st != PW_OK) return st;
  st = launch_combine(ctx, T, top_k, ksplit, out, stream);
  if (st != PW_OK) return st;
  st = launch_observe(ctx, layer, T, top_k, stream);
  ctx->last_T = T;
  ctx->last_k = top_k;
  return st;
}

extern "C" pw_status pw_moe_forward_host(pw_ctx* ctx, int layer, const void* hidden_host, const float* logits_host, int T,
                                         int top_k, float* out_host, pw_mode mode, pw_stream stream) {
  if (!ctx || !hidden_host || !logits_host || !out_host) return PW_ERR_INVALID_ARG;
  const pw_config& c = ctx->cfg;
  if (T < 1 || T > c.max_tokens) return PW_ERR_INVALID_ARG;
  char* b = ctx->base;
  const WsMap& w = ctx->ws;
  // refuse what the forward call would refuse before the first copy is enqueued (the staging buffers stay untouched)
  const pw_status as = check_forward_args(ctx, layer, b + w.io_hidden, reinterpret_cast<const float*>(b + w.io_logits), T,
                                          top_k, nullptr, reinterpret_cast<const float*>(b + w.io_out), mode);
  if (as != PW_OK) return as;
  PW_CUDA_OK(cudaMemcpyAsync(b + w.io_hidden, hidden_host, (size_t)T * c.hidden * 2, cudaMemcpyHostToDevice, stream));
  PW_CUDA_OK(cudaMemcpyAsync(b + w.io_logits, logits_host, (size_t)T * c.n_experts * 4, cudaMemcpyHostToDevice, stream));
  pw_status st = pw_moe_forward(ctx, layer, b + w.io_hidden, reinterpret_cast<const float*>(b + w.io_logits), T, top_k,
                                nullptr, reinterpret_cast<float*>(b + w.io_out), mode, stream);
  if (st != PW_OK) return st;
  PW_CUDA_OK(cudaMemcpyAsync(out_host, b + w.io_out, (size_t)T * c.hidden * 4, cudaMemcpyDeviceToHost, stream));
  return PW_OK;
}

extern "C" pw_status pw_get_routing(pw_ctx* ctx, int32_t* topk_ids, float* gates, int32_t* counts, int32_t* offsets,
                                    int32_t* perm, pw_stream stream) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  if (ctx->last_T == 0) return PW_ERR_STATE;
  const size_t P = (size_t)ctx->last_T * ctx->last_k;
  const int E = ctx->cfg.n_experts;
  char* b = ctx->base;
  const WsMap& w = ctx->ws;
  if (topk_ids) PW_CUDA_OK(cudaMemcpyAsync(topk_ids, b + w.topk_ids, 4 * P, cudaMemcpyDeviceToDevice, stream));
  if (gates) PW_CUDA_OK(cudaMemcpyAsync(gates, b + w.gates, 4 * P, cudaMemcpyDeviceToDevice, stream));
  if (counts) PW_CUDA_OK(cudaMemcpyAsync(counts, b + w.counts, 4 * (size_t)E, cudaMemcpyDeviceToDevice, stream));
  if (offsets) PW_CUDA_OK(cudaMemcpyAsync(offsets, b + w.offsets, 4 * (size_t)(E + 1), cudaMemcpyDeviceToDevice, stream));
  if (perm) PW_CUDA_OK(cudaMemcpyAsync(perm, b + w.perm, 4 * P, cudaMemcpyDeviceToDevice, stream));
  return PW_OK;
}

extern "C" pw_status pw_last_device_status(pw_ctx* ctx) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  int32_t v = 0;
  PW_CUDA_OK(cudaDeviceSynchronize());
  PW_CUDA_OK(cudaMemcpy(&v, ctx->base + ctx->ws.status, 4, cudaMemcpyDeviceToHost));
  if (v != 0) {
    PW_CUDA_OK(cudaMemset(ctx->base + ctx->ws.status, 0, 4));
  }
  return (pw_status)v;
}

extern "C" pw_status pw_kernel_timing(pw_ctx* ctx, int enable) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  if (enable && !ctx->timing_ev) {
    const int n = pw_ctx::kTimingSlots * (PW_NUM_KERNELS + 1);
    ctx->timing_ev = new (std::nothrow) cudaEvent_t[n]();
    if (!ctx->timing_ev) return PW_ERR_NOMEM;
    for (int i = 0; i < n; ++i) PW_CUDA_OK(cudaEventCreate(&ctx->timing_ev[i]));
  }
  if (ctx->timing_ev)
    for (int i = 0; i < pw_ctx::kTimingSlots; ++i) timing_drain_slot(ctx, i);
  ctx->timing_on = enable != 0;
  if (enable) {
    ctx->timing_calls = 0;
    for (int i = 0; i < PW_NUM_KERNELS; ++i) ctx->timing_ms[i] = 0.0;
  }
  return PW_OK;
}

extern "C" pw_status pw_get_kernel_times(pw_ctx* ctx, double* ms_out, uint64_t* calls_out) {
  if (!ctx || !ms_out) return PW_ERR_INVALID_ARG;
  if (ctx->timing_ev)
    for (int i = 0; i < pw_ctx::kTimingSlots; ++i) timing_drain_slot(ctx, i);
  for (int i = 0; i < PW_NUM_KERNELS; ++i) ms_out[i] = ctx->timing_ms[i];
  if (calls_out) *calls_out = ctx->timing_calls;
  return PW_OK;
}

extern "C" pw_status pw_debug_set_wait(pw_ctx* ctx, uint32_t polls, uint32_t hook) {
  if (!ctx) return PW_ERR_INVALID_ARG;
  ctx->wait_polls = polls;
  ctx->test_hook = hook;
  return PW_OK;
}

extern "C" uint64_t pw_launch_count(pw_ctx* ctx) { return ctx ? ctx->launches : 0; }

extern "C" const char* pw_status_str(pw_status s) {
  switch (s) {
    case PW_OK: return "ok";
    case PW_ERR_INVALID_ARG: return "invalid argument";
    case PW_ERR_SHAPE: return "bad shape";
    case PW_ERR_BITS: return "bad bitwidth";
    case PW_ERR_ALIGN: return "misaligned pointer";
    case PW_ERR_STATE: return "bad state";
    case PW_ERR_NOMEM: return "workspace too small";
    case PW_ERR_CUDA: return "CUDA error";
    case PW_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown";
}
