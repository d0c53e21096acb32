// extern "C" entry points of libtreelstm_b200 (declared in include/treelstm.h): argument checks,
// parameter copies, workspace layout and the launch sequence of one forward / backward call.
#include <new>

#include "common.cuh"

namespace tl {

WsLayout ws_layout(const treelstm* ctx, int n, bool with_backward) {
  WsLayout L{};
  const size_t nn = n < 1 ? 1 : (size_t)n;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up_sz(bytes, 256); return o; };
  L.status = take(sizeof(DevStatus));
  L.parent = take(4 * nn);
  L.pending = take(4 * nn);
  L.order_tmp = take(4 * nn);
  L.level_offset = take(4 * (nn + 2));
  L.roots = take(4 * nn);
  L.table = take(4 * (size_t)kRadixBins * ((nn + kRadixChunk - 1) / kRadixChunk));
  L.slot = take(4 * nn);
  L.part_order = L.part_offset = L.part_spill = L.xin = L.ain = L.cin = off;
  if (ctx->precision == TREELSTM_BF16) {
    L.part_order = take(4 * nn);                     // node ids by (sub-forest, level, id)
    L.part_offset = take(4 * (kMaxParts + 1));
    L.part_spill = take(4 * (nn + kMaxParts + 1));   // wavefront boundaries of very deep sub-forests
    L.xin = take(2 * nn * (size_t)ctx->Ep);          // leaf embedding rows in ready order
    L.ain = take(2 * nn * 2 * (size_t)ctx->Hp);      // [h_l | h_r] of every position, bf16
    L.cin = take(4 * nn * 2 * (size_t)ctx->H);       // [c_l | c_r] of every position, fp32
    L.pre = take(4 * 1024);                          // leaves per CTA (wavefront kernel started under the scheduler)
  }
  L.gates = L.dh = L.dc = L.dz = L.tok_slot = off;
  if (with_backward) {
    const size_t H = (size_t)ctx->H;
    L.gates = take(4 * nn * 5 * H);
    L.dh = take(4 * nn * H);
    L.dc = take(4 * nn * H);
    L.dz = take(4 * nn * 5 * H);
    L.tok_slot = take(4 * ((size_t)ctx->vocab + 4 + ((size_t)ctx->vocab + 127) / 128));   // vocab + 1 entries in use, the scan
                                                                   // reads whole quads; then one count per 128 ids
  }
  L.trace = off;
#ifdef TREELSTM_TRACE
  L.trace = take(2 * sizeof(long long) * kTraceSlots * kTraceLevels);   // grid kernel | cluster kernel
#endif
  L.check = off;
#ifdef TREELSTM_CHECKED
  L.check = take(3 * 4 * nn);
#endif
  L.total = off;
  return L;
}

namespace {

int copy_params(treelstm* ctx, const float* emb, const float* W, const float* b, cudaStream_t s) {
  const size_t H = ctx->H, E = ctx->E, V = ctx->vocab;
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->emb, emb, sizeof(float) * V * E, cudaMemcpyDeviceToDevice, s));
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->W, W, sizeof(float) * (E + 2 * H) * 5 * H, cudaMemcpyDeviceToDevice, s));
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->b, b, sizeof(float) * 5 * H, cudaMemcpyDeviceToDevice, s));
  if (ctx->precision == TREELSTM_BF16) {
    int rc = pack_weights_bf16(ctx, s);
    if (rc != TREELSTM_OK) return rc;
  }
  TL_CUDA(ctx, cudaStreamSynchronize(s));
  return TREELSTM_OK;
}

void free_host_path(treelstm* ctx) {
  auto& p = ctx->hp;
  if (p.owned) {
    cudaFree(p.forest); cudaFree(p.level); cudaFree(p.order);
    cudaFree(p.n_levels); cudaFree(p.roots_pack); cudaFree(p.n_roots); cudaFree(p.h); cudaFree(p.c);
    cudaFree(p.ws);
  }
  unsigned char* ext = p.ext;
  const size_t ext_bytes = p.ext_bytes;
  p = treelstm::HostPath{};
  p.ext = ext; p.ext_bytes = ext_bytes;
}

// Device staging of treelstm_forward_host for forests of up to `cap` nodes: offsets of its parts in
// one buffer (every part 256-byte aligned) and the total.
struct HostStaging {
  size_t forest, level, order, n_levels, roots_pack, n_roots, h, c, ws, ws_bytes, total;
};
HostStaging host_staging_layout(const treelstm* ctx, size_t cap) {
  HostStaging L{};
  const size_t H = ctx->H;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += round_up_sz(bytes, 256); return o; };
  L.forest = take(12 * cap);
  L.level = take(4 * cap);
  L.order = take(4 * cap);
  L.n_levels = take(256);
  L.roots_pack = take((4 + 8 * H) * cap);
  L.n_roots = take(256);
  L.h = take(4 * cap * H);
  L.c = take(4 * cap * H);
  L.ws_bytes = ws_layout(ctx, (int)cap, false).total;
  L.ws = take(L.ws_bytes);
  L.total = off;
  return L;
}

// True if the calling thread's current device is the one the context was created on.
bool on_own_device(const treelstm* ctx) {
  int dev = -1;
  return cudaGetDevice(&dev) == cudaSuccess && dev == ctx->device;
}

// Read the control block and the level table back (one synchronisation).
int read_levels(treelstm* ctx) {
  auto& L = ctx->last;
  char* base = static_cast<char*>(L.ws);
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->host_status, base + L.lay.status, sizeof(DevStatus),
                               cudaMemcpyDeviceToHost, L.stream));
  // the level table is at most (n + 1) / 2 + 1 entries; small forests are copied whole, large
  // ones after the count is known
  const int quick = 4096;
  int cap_needed = L.n + 2 < quick ? L.n + 2 : quick;
  if (ctx->host_level_cap < cap_needed || !ctx->host_level_offset) {
    if (ctx->host_level_offset) cudaFreeHost(ctx->host_level_offset);
    ctx->host_level_offset = nullptr;
    TL_CUDA(ctx, cudaMallocHost((void**)&ctx->host_level_offset, sizeof(int32_t) * cap_needed));
    ctx->host_level_cap = cap_needed;
  }
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->host_level_offset, L.level_offset, sizeof(int32_t) * cap_needed,
                               cudaMemcpyDeviceToHost, L.stream));
  TL_CUDA(ctx, cudaStreamSynchronize(L.stream));
  const DevStatus* hs = reinterpret_cast<const DevStatus*>(ctx->host_status);
  if (hs->status != 0) return hs->status;
  const int n_levels = hs->n_levels;
  if (n_levels + 1 > cap_needed) {
    cudaFreeHost(ctx->host_level_offset);
    ctx->host_level_offset = nullptr;
    TL_CUDA(ctx, cudaMallocHost((void**)&ctx->host_level_offset, sizeof(int32_t) * (n_levels + 1)));
    ctx->host_level_cap = n_levels + 1;
    TL_CUDA(ctx, cudaMemcpyAsync(ctx->host_level_offset, L.level_offset,
                                 sizeof(int32_t) * (n_levels + 1), cudaMemcpyDeviceToHost, L.stream));
    TL_CUDA(ctx, cudaStreamSynchronize(L.stream));
  }
  L.n_levels = n_levels;
  L.host_levels_valid = true;
  return TREELSTM_OK;
}

}  // namespace

// What a control block that has just been read back says about the hand-over to the cluster kernel.
void learn_tail_hint(treelstm* ctx) {
  const DevStatus* hs = reinterpret_cast<const DevStatus*>(ctx->host_status);
  const auto& L = ctx->last;
  if (!ctx->tail_ok || ctx->precision != TREELSTM_BF16 || L.mode != TREELSTM_PERSISTENT || hs->status != 0 || hs->n_levels <= 0)
    return;
  ctx->tail_skip = hs->tail_from >= hs->n_levels;
}

// used by backward.cu
int ensure_host_levels(treelstm* ctx) {
  if (ctx->last.host_levels_valid) return TREELSTM_OK;
  return read_levels(ctx);
}

}  // namespace tl

using namespace tl;

extern "C" {

int treelstm_create(treelstm_t** out, int H, int E, int vocab, const float* emb, const float* W,
                    const float* b, int precision, void* stream) {
  if (!out) return TREELSTM_ERR_INVALID_ARG;
  *out = nullptr;
  if (H <= 0 || E <= 0 || vocab <= 0 || !emb || !W || !b) return TREELSTM_ERR_INVALID_ARG;
  if (precision != TREELSTM_FP32 && precision != TREELSTM_BF16) return TREELSTM_ERR_INVALID_ARG;
  if (H > 8192 || E > 8192) return TREELSTM_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TREELSTM_ERR_NO_DEVICE;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return TREELSTM_ERR_NO_DEVICE;
  if (prop.major != 10) return TREELSTM_ERR_NO_DEVICE;  // kernels are built for sm_100a only
  treelstm* ctx = new (std::nothrow) treelstm();
  if (!ctx) return TREELSTM_ERR_INVALID_ARG;
  ctx->H = H; ctx->E = E; ctx->vocab = vocab; ctx->precision = precision;
  ctx->Hp = round_up(H, kKBlock);
  ctx->Ep = round_up(E, kKBlock);
  ctx->device = dev;
  ctx->sm_count = prop.multiProcessorCount;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t Hs = H, Es = E, V = vocab;
  auto fail = [&](int rc) { treelstm_destroy(ctx); return rc; };
  if (cudaMalloc((void**)&ctx->emb, sizeof(float) * V * Es) != cudaSuccess ||
      cudaMalloc((void**)&ctx->W, sizeof(float) * (Es + 2 * Hs) * 5 * Hs) != cudaSuccess ||
      cudaMalloc((void**)&ctx->b, sizeof(float) * 5 * Hs) != cudaSuccess ||
      cudaMallocHost((void**)&ctx->host_status, sizeof(DevStatus)) != cudaSuccess)
    return fail(TREELSTM_ERR_CUDA);
  if (precision == TREELSTM_BF16) {
    const size_t Hp = ctx->Hp, Ep = ctx->Ep, groups = Hp / kUnitGroup;
    if (cudaMalloc((void**)&ctx->emb_bf, 2 * V * Ep) != cudaSuccess ||
        cudaMalloc((void**)&ctx->Wp_h, 2 * groups * 40 * 2 * Hp) != cudaSuccess ||
        cudaMalloc((void**)&ctx->Wp_x, 2 * groups * 24 * Ep) != cudaSuccess ||
        cudaMalloc((void**)&ctx->bp_h, 4 * groups * 40) != cudaSuccess ||
        cudaMalloc((void**)&ctx->bp_x, 4 * groups * 24) != cudaSuccess)
      return fail(TREELSTM_ERR_CUDA);
  }
  int rc = init_schedule_attributes(ctx);
  if (rc == TREELSTM_OK && precision == TREELSTM_BF16) rc = init_tc_attributes(ctx);
  if (rc == TREELSTM_OK) rc = init_dweight_tc_attributes(ctx);
  if (rc != TREELSTM_OK) return fail(rc);
  rc = copy_params(ctx, emb, W, b, s);
  if (rc != TREELSTM_OK) return fail(rc);
  ctx->sf = subforest_plan(ctx);
  ctx->tail_ok = ctx->sf.ok && init_tail_attributes(ctx) == TREELSTM_OK;
  *out = ctx;
  return TREELSTM_OK;
}

int treelstm_create_recursive(treelstm_t** out, int cell, int H, int vocab, const float* emb, const float* W,
                              const float* b, const float* V, void* stream) {
  if (!out) return TREELSTM_ERR_INVALID_ARG;
  *out = nullptr;
  if (cell != TREELSTM_CELL_TREERNN && cell != TREELSTM_CELL_RNTN) return TREELSTM_ERR_INVALID_ARG;
  if (H <= 0 || vocab <= 0 || !emb || !W || !b || (cell == TREELSTM_CELL_RNTN && !V)) return TREELSTM_ERR_INVALID_ARG;
  if (H > 4096 || (cell == TREELSTM_CELL_RNTN && H > 128)) return TREELSTM_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TREELSTM_ERR_NO_DEVICE;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return TREELSTM_ERR_NO_DEVICE;
  if (prop.major != 10) return TREELSTM_ERR_NO_DEVICE;
  treelstm* ctx = new (std::nothrow) treelstm();
  if (!ctx) return TREELSTM_ERR_INVALID_ARG;
  ctx->H = H; ctx->E = H; ctx->vocab = vocab; ctx->precision = TREELSTM_FP32; ctx->cell = cell;
  ctx->Hp = round_up(H, kKBlock); ctx->Ep = ctx->Hp;
  ctx->device = dev;
  ctx->sm_count = prop.multiProcessorCount;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t Hs = H, V_ = vocab, K2 = 2 * Hs, KQ = cell == TREELSTM_CELL_RNTN ? K2 * K2 : 0;
  auto fail = [&](int rc) { treelstm_destroy(ctx); return rc; };
  if (cudaMalloc((void**)&ctx->emb, sizeof(float) * V_ * Hs) != cudaSuccess ||
      cudaMalloc((void**)&ctx->Wcat, sizeof(float) * (KQ + K2) * Hs) != cudaSuccess ||
      cudaMalloc((void**)&ctx->b, sizeof(float) * Hs) != cudaSuccess ||
      cudaMallocHost((void**)&ctx->host_status, sizeof(DevStatus)) != cudaSuccess)
    return fail(TREELSTM_ERR_CUDA);
  int rc = init_schedule_attributes(ctx);
  if (rc != TREELSTM_OK) return fail(rc);
  if (cudaMemcpyAsync(ctx->emb, emb, sizeof(float) * V_ * Hs, cudaMemcpyDeviceToDevice, s) != cudaSuccess ||
      cudaMemcpyAsync(ctx->b, b, sizeof(float) * Hs, cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return fail(TREELSTM_ERR_CUDA);
  rc = pack_weights_rec(ctx, W, V, s);
  if (rc != TREELSTM_OK) return fail(rc);
  if (cudaStreamSynchronize(s) != cudaSuccess) return fail(TREELSTM_ERR_CUDA);
  *out = ctx;
  return TREELSTM_OK;
}

int treelstm_update_weights(treelstm_t* ctx, const float* emb, const float* W, const float* b,
                            void* stream) {
  if (!ctx || !emb || !W || !b) return TREELSTM_ERR_INVALID_ARG;
  if (ctx->cell != 0) return TREELSTM_ERR_UNSUPPORTED;   // TreeRNN / RNTN contexts are created anew
  return copy_params(ctx, emb, W, b, static_cast<cudaStream_t>(stream));
}

int treelstm_set_classifier(treelstm_t* ctx, int C, const float* Wc, const float* bc, void* stream) {
  if (!ctx || !Wc || !bc || C < 1) return TREELSTM_ERR_INVALID_ARG;
  if (C > 32) return TREELSTM_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaFree(ctx->Wc); cudaFree(ctx->bc);
  ctx->Wc = ctx->bc = nullptr; ctx->C = 0;
  TL_CUDA(ctx, cudaMalloc((void**)&ctx->Wc, sizeof(float) * ctx->H * C));
  TL_CUDA(ctx, cudaMalloc((void**)&ctx->bc, sizeof(float) * C));
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->Wc, Wc, sizeof(float) * ctx->H * C, cudaMemcpyDeviceToDevice, s));
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->bc, bc, sizeof(float) * C, cudaMemcpyDeviceToDevice, s));
  TL_CUDA(ctx, cudaStreamSynchronize(s));
  ctx->C = C;
  return TREELSTM_OK;
}

int treelstm_set_option(treelstm_t* ctx, int key, long long value) {
  if (!ctx || value < 0) return TREELSTM_ERR_INVALID_ARG;
  switch (key) {
    case TREELSTM_OPT_SCHED_SINGLE_CTA_MAX:
      ctx->opt.sched_single_cta_max = value > kSchedSingleMaxNodes ? kSchedSingleMaxNodes : (int)value;
      return TREELSTM_OK;
    case TREELSTM_OPT_WAIT_LIMIT_CYCLES:
      if (value < 1 || value > (1ll << 24)) return TREELSTM_ERR_INVALID_ARG;
      ctx->opt.wait_limit_kcycles = value;
      return TREELSTM_OK;
    case TREELSTM_OPT_MAX_CTAS:
      ctx->opt.max_ctas = value > 65535 ? 65535 : (int)value;
      return TREELSTM_OK;
    case TREELSTM_OPT_TAIL_WIDTH:
      ctx->opt.tail_width = value > 64 ? 64 : (int)value;
      ctx->tail_skip = false;
      return TREELSTM_OK;
    case TREELSTM_OPT_TAIL_MIN_LEVELS:
      ctx->opt.tail_min_levels = value > (1 << 20) ? (1 << 20) : (int)value;
      ctx->tail_skip = false;
      return TREELSTM_OK;
    case TREELSTM_OPT_LEAVES_FIRST_MIN_NODES:
      ctx->opt.leaves_first_min_nodes = value > (1 << 30) ? (1 << 30) : (int)value;
      return TREELSTM_OK;
    case TREELSTM_OPT_OVERLAP_LAUNCH:
      ctx->opt.overlap_launch = value != 0;
      return TREELSTM_OK;
    case TREELSTM_OPT_DW_TENSOR_CORES:
      ctx->opt.dw_tensor_cores = value != 0;
      return TREELSTM_OK;
    case TREELSTM_OPT_TAIL_MAX_NODES:
      ctx->opt.tail_max_nodes = value > (1 << 30) ? (1 << 30) : (int)value;
      return TREELSTM_OK;
    case TREELSTM_OPT_TIME_WAVEFRONT_KERNEL:
      if (value && !ctx->ev_begin) {
        TL_CUDA(ctx, cudaEventCreate(&ctx->ev_begin));
        TL_CUDA(ctx, cudaEventCreate(&ctx->ev_end));
      }
      ctx->opt.time_kernel = value != 0;
      return TREELSTM_OK;
    default:
      return TREELSTM_ERR_INVALID_ARG;
  }
}

size_t treelstm_workspace_bytes(const treelstm_t* ctx, int max_nodes, int with_backward) {
  if (!ctx || max_nodes < 0) return 0;
  return ws_layout(ctx, max_nodes, with_backward != 0).total;
}

int treelstm_forward(treelstm_t* ctx, int n_nodes, const int32_t* left, const int32_t* right,
                     const int32_t* token, float* h, float* c, int32_t* level, int32_t* order,
                     int32_t* level_offset, int32_t* n_levels, int flags, void* workspace,
                     size_t workspace_bytes, void* stream) {
  if (!ctx) return TREELSTM_ERR_INVALID_ARG;
  ctx->last.valid = false;
  ctx->launches = 0;
  if (!on_own_device(ctx)) return TREELSTM_ERR_STATE;
  if (n_nodes < 0 || !n_levels || !workspace) return TREELSTM_ERR_INVALID_ARG;
  if (n_nodes > 0 && (!left || !right || !token || !h || (!c && ctx->cell == 0) || !level || !order))
    return TREELSTM_ERR_INVALID_ARG;
  if (flags & ~(TREELSTM_PERSISTENT | TREELSTM_SAVE_FOR_BACKWARD | TREELSTM_SUBFORESTS)) return TREELSTM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return TREELSTM_ERR_INVALID_ARG;
  const bool save = (flags & TREELSTM_SAVE_FOR_BACKWARD) != 0;
  const WsLayout lay = ws_layout(ctx, n_nodes, save);
  if (workspace_bytes < lay.total) return TREELSTM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  char* base = static_cast<char*>(workspace);
  int32_t* lvl_off = level_offset ? level_offset : reinterpret_cast<int32_t*>(base + lay.level_offset);

  auto& L = ctx->last;
  L.n = n_nodes; L.flags = flags; L.left = left; L.right = right; L.token = token;
  L.h = h; L.c = c; L.level = level; L.order = order; L.level_offset = lvl_off;
  L.ws = workspace; L.lay = lay; L.stream = s; L.host_levels_valid = false; L.n_levels = 0;

  // Sub-forest mode needs the cluster plan of this context and a forest the single-CTA scheduler
  // can deal out; anything else runs the grid-wide persistent kernel instead.
  const int single_max = ctx->opt.sched_single_cta_max < kSchedPartMaxNodes ? ctx->opt.sched_single_cta_max
                                                                             : kSchedPartMaxNodes;
  const bool subforests = (flags & TREELSTM_SUBFORESTS) && ctx->precision == TREELSTM_BF16 && ctx->sf.ok &&
                          n_nodes > 0 && n_nodes <= single_max;
  int rc = launch_schedule(ctx, n_nodes, left, right, token, level, order, lvl_off, n_levels, workspace,
                           lay, subforests ? ctx->sf.n_parts : 0, s);
  if (rc != TREELSTM_OK) return rc;
  const bool persistent = (flags & (TREELSTM_PERSISTENT | TREELSTM_SUBFORESTS)) != 0;
  L.mode = subforests ? TREELSTM_SUBFORESTS : (persistent ? TREELSTM_PERSISTENT : TREELSTM_PER_LEVEL);
  L.valid = true;
  if (n_nodes == 0) return TREELSTM_OK;

  if (!persistent) {
    rc = read_levels(ctx);
    if (rc != TREELSTM_OK) { L.valid = false; return rc; }
  }
  rc = launch_check_clear(ctx, n_nodes, workspace, lay, s);
  if (rc != TREELSTM_OK) { L.valid = false; return rc; }
  ctx->ev_valid = false;
  if (ctx->opt.time_kernel) TL_CUDA(ctx, cudaEventRecord(ctx->ev_begin, s));
  if (ctx->cell != 0)
    rc = launch_forward_rec(ctx, n_nodes, left, right, token, h, order, lvl_off, ctx->host_level_offset, L.n_levels,
                            persistent ? (flags | TREELSTM_PERSISTENT) : flags, workspace, lay, s);
  else if (subforests)
    rc = launch_forward_bf16_subforest(ctx, n_nodes, left, right, token, h, c, level, flags, workspace, lay, s);
  else if (ctx->precision == TREELSTM_BF16)
    rc = launch_forward_bf16(ctx, n_nodes, left, right, token, h, c, order, lvl_off,
                             ctx->host_level_offset, L.n_levels, persistent ? (flags | TREELSTM_PERSISTENT) : flags,
                             workspace, lay, s);
  else
    rc = launch_forward_fp32(ctx, n_nodes, left, right, token, h, c, order, lvl_off,
                             ctx->host_level_offset, L.n_levels, persistent ? (flags | TREELSTM_PERSISTENT) : flags,
                             workspace, lay, s);
  if (ctx->opt.time_kernel && rc == TREELSTM_OK) {
    TL_CUDA(ctx, cudaEventRecord(ctx->ev_end, s));
    ctx->ev_valid = true;
  }
  if (rc == TREELSTM_OK)
    rc = launch_check_counts(ctx, n_nodes, subforests ? reinterpret_cast<const int32_t*>(base + lay.part_order) : order,
                             left, workspace, lay, s);
  if (rc != TREELSTM_OK) L.valid = false;
  return rc;
}

int treelstm_last_kernel_ms(treelstm_t* ctx, float* ms) {
  if (!ctx || !ms) return TREELSTM_ERR_INVALID_ARG;
  if (!ctx->ev_valid) return TREELSTM_ERR_STATE;
  TL_CUDA(ctx, cudaEventSynchronize(ctx->ev_end));
  TL_CUDA(ctx, cudaEventElapsedTime(ms, ctx->ev_begin, ctx->ev_end));
  return TREELSTM_OK;
}

int treelstm_status_sync(treelstm_t* ctx) {
  if (!ctx) return TREELSTM_ERR_INVALID_ARG;
  auto& L = ctx->last;
  if (!L.ws) return TREELSTM_ERR_STATE;
  char* base = static_cast<char*>(L.ws);
  TL_CUDA(ctx, cudaMemcpyAsync(ctx->host_status, base + L.lay.status, sizeof(DevStatus),
                               cudaMemcpyDeviceToHost, L.stream));
  TL_CUDA(ctx, cudaStreamSynchronize(L.stream));
  const int st = reinterpret_cast<const DevStatus*>(ctx->host_status)->status;
  if (st != 0) L.valid = false;
  else learn_tail_hint(ctx);
  return st;
}

int treelstm_roots(treelstm_t* ctx, int max_roots, int32_t* root_ids, float* root_h, float* root_c,
                   int32_t* n_roots, void* stream) {
  if (!ctx || max_roots < 0 || !n_roots) return TREELSTM_ERR_INVALID_ARG;
  if (!ctx->last.valid) return TREELSTM_ERR_STATE;
  return launch_gather_roots(ctx, max_roots, root_ids, root_h, root_c, n_roots,
                             static_cast<cudaStream_t>(stream));
}

int treelstm_backward(treelstm_t* ctx, const int32_t* labels, float* loss, float* dW, float* db,
                      float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows,
                      int32_t* n_touched, void* stream) {
  if (!ctx || !labels || !loss || !dW || !db || !dWc || !dbc || !touched_ids || !dEmb_rows ||
      !n_touched)
    return TREELSTM_ERR_INVALID_ARG;
  if (!ctx->last.valid || !(ctx->last.flags & TREELSTM_SAVE_FOR_BACKWARD) || ctx->C < 1)
    return TREELSTM_ERR_STATE;
  if (ctx->cell != 0) return TREELSTM_ERR_STATE;   // TreeRNN / RNTN contexts: treelstm_backward_recursive
  if (!on_own_device(ctx)) return TREELSTM_ERR_STATE;
  ctx->launches = 0;
  return launch_backward(ctx, labels, loss, dW, db, dWc, dbc, touched_ids, dEmb_rows, n_touched,
                         static_cast<cudaStream_t>(stream));
}

int treelstm_backward_recursive(treelstm_t* ctx, const int32_t* labels, float* loss, float* dW, float* db, float* dV,
                                float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows,
                                int32_t* n_touched, void* stream) {
  if (!ctx || !labels || !loss || !dW || !db || !dWc || !dbc || !touched_ids || !dEmb_rows || !n_touched)
    return TREELSTM_ERR_INVALID_ARG;
  if (ctx->cell == 0) return TREELSTM_ERR_STATE;
  if (ctx->cell == TREELSTM_CELL_RNTN && !dV) return TREELSTM_ERR_INVALID_ARG;
  if (!ctx->last.valid || !(ctx->last.flags & TREELSTM_SAVE_FOR_BACKWARD) || ctx->C < 1)
    return TREELSTM_ERR_STATE;
  if (!on_own_device(ctx)) return TREELSTM_ERR_STATE;
  ctx->launches = 0;
  return launch_backward_rec(ctx, labels, loss, dW, db, dV, dWc, dbc, touched_ids, dEmb_rows, n_touched,
                             static_cast<cudaStream_t>(stream));
}

int treelstm_forward_host(treelstm_t* ctx, int n_nodes, const int32_t* left, const int32_t* right,
                          const int32_t* token, float* h, float* c, int32_t* level, int32_t* order,
                          int32_t* n_levels, int max_roots, int32_t* root_ids, float* root_h,
                          float* root_c, int32_t* n_roots, int flags, void* stream) {
  if (!ctx || n_nodes < 0 || max_roots < 0) return TREELSTM_ERR_INVALID_ARG;
  if (n_nodes > 0 && (!left || !right || !token)) return TREELSTM_ERR_INVALID_ARG;
  if (flags & TREELSTM_SAVE_FOR_BACKWARD) return TREELSTM_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (!on_own_device(ctx)) return TREELSTM_ERR_STATE;
  auto& p = ctx->hp;
  const size_t H = ctx->H;
  if (p.ext) {
    // the caller's staging memory: carved up anew whenever the forest outgrows the last carving
    if (n_nodes > p.cap_nodes || !p.ws || p.owned) {
      const size_t cap = n_nodes < 1 ? 1 : (size_t)n_nodes;
      const HostStaging L = host_staging_layout(ctx, cap);
      if (L.total > p.ext_bytes) return TREELSTM_ERR_INVALID_ARG;
      free_host_path(ctx);
      unsigned char* b = p.ext;
      p.forest = reinterpret_cast<int32_t*>(b + L.forest);
      p.level = reinterpret_cast<int32_t*>(b + L.level);
      p.order = reinterpret_cast<int32_t*>(b + L.order);
      p.n_levels = reinterpret_cast<int32_t*>(b + L.n_levels);
      p.roots_pack = b + L.roots_pack;
      p.n_roots = reinterpret_cast<int32_t*>(b + L.n_roots);
      p.h = reinterpret_cast<float*>(b + L.h);
      p.c = reinterpret_cast<float*>(b + L.c);
      p.ws = b + L.ws;
      p.ws_bytes = L.ws_bytes;
      p.cap_nodes = (int)cap;
      p.owned = false;
    }
  } else if (n_nodes > p.cap_nodes || !p.ws) {
    free_host_path(ctx);
    const size_t cap = n_nodes < 1024 ? 1024 : (size_t)n_nodes + n_nodes / 4;
    p.ws_bytes = ws_layout(ctx, (int)cap, false).total;
    p.owned = true;
    // the three forest arrays share one buffer, the root outputs another: when the caller's host
    // arrays are adjacent in the same way, each group moves in a single copy
    if (cudaMalloc((void**)&p.forest, 12 * cap) != cudaSuccess || cudaMalloc((void**)&p.level, 4 * cap) != cudaSuccess ||
        cudaMalloc((void**)&p.order, 4 * cap) != cudaSuccess || cudaMalloc((void**)&p.n_levels, 256) != cudaSuccess ||
        cudaMalloc((void**)&p.roots_pack, (4 + 8 * H) * cap) != cudaSuccess || cudaMalloc((void**)&p.n_roots, 256) != cudaSuccess ||
        cudaMalloc((void**)&p.h, 4 * cap * H) != cudaSuccess || cudaMalloc((void**)&p.c, 4 * cap * H) != cudaSuccess ||
        cudaMalloc(&p.ws, p.ws_bytes) != cudaSuccess) {
      ctx->cuda_error = (int)cudaGetLastError();
      free_host_path(ctx);
      return TREELSTM_ERR_CUDA;
    }
    p.cap_nodes = (int)cap;
  }
  const size_t nb = 4 * (size_t)n_nodes;
  p.left = p.forest; p.right = p.forest + n_nodes; p.token = p.forest + 2 * (size_t)n_nodes;
  if (n_nodes > 0) {
    if (right == left + n_nodes && token == right + n_nodes) {
      TL_CUDA(ctx, cudaMemcpyAsync(p.left, left, 3 * nb, cudaMemcpyHostToDevice, s));
    } else {
      TL_CUDA(ctx, cudaMemcpyAsync(p.left, left, nb, cudaMemcpyHostToDevice, s));
      TL_CUDA(ctx, cudaMemcpyAsync(p.right, right, nb, cudaMemcpyHostToDevice, s));
      TL_CUDA(ctx, cudaMemcpyAsync(p.token, token, nb, cudaMemcpyHostToDevice, s));
    }
  }
  int rc = treelstm_forward(ctx, n_nodes, p.left, p.right, p.token, p.h, p.c, p.level, p.order, nullptr,
                            p.n_levels, flags, p.ws, p.ws_bytes, s);
  if (rc != TREELSTM_OK) return rc;
  const int launches_fwd = ctx->launches;
  const bool want_roots = root_ids || root_h || root_c || n_roots;
  int max_r = max_roots < n_nodes ? max_roots : n_nodes;
  p.root_ids = reinterpret_cast<int32_t*>(p.roots_pack);
  p.root_h = reinterpret_cast<float*>(p.root_ids + max_r);
  p.root_c = p.root_h + (size_t)max_r * H;
  if (want_roots) {
    rc = launch_gather_roots(ctx, max_r, p.root_ids, p.root_h, p.root_c, p.n_roots, s);
    if (rc != TREELSTM_OK) return rc;
  }
  if (n_nodes > 0) {
    if (h) TL_CUDA(ctx, cudaMemcpyAsync(h, p.h, nb * H, cudaMemcpyDeviceToHost, s));
    if (c && ctx->cell == 0) TL_CUDA(ctx, cudaMemcpyAsync(c, p.c, nb * H, cudaMemcpyDeviceToHost, s));
    if (level) TL_CUDA(ctx, cudaMemcpyAsync(level, p.level, nb, cudaMemcpyDeviceToHost, s));
    if (order) TL_CUDA(ctx, cudaMemcpyAsync(order, p.order, nb, cudaMemcpyDeviceToHost, s));
  }
  if (want_roots && max_r > 0) {
    // the number of roots is not known on the host yet: copy max_r rows (rows past n_roots are
    // unspecified) - callers pass the number of trees they submitted
    if (root_ids && root_h && root_c && max_r == max_roots &&
        root_h == reinterpret_cast<float*>(root_ids + max_r) && root_c == root_h + (size_t)max_r * H) {
      TL_CUDA(ctx, cudaMemcpyAsync(root_ids, p.root_ids, (4 + 8 * H) * (size_t)max_r, cudaMemcpyDeviceToHost, s));
    } else {
      if (root_ids) TL_CUDA(ctx, cudaMemcpyAsync(root_ids, p.root_ids, 4 * (size_t)max_r, cudaMemcpyDeviceToHost, s));
      if (root_h) TL_CUDA(ctx, cudaMemcpyAsync(root_h, p.root_h, 4 * (size_t)max_r * H, cudaMemcpyDeviceToHost, s));
      if (root_c) TL_CUDA(ctx, cudaMemcpyAsync(root_c, p.root_c, 4 * (size_t)max_r * H, cudaMemcpyDeviceToHost, s));
    }
  }
  // the level and root counts come back with the control block that the status read copies anyway
  rc = treelstm_status_sync(ctx);
  const DevStatus* hs = reinterpret_cast<const DevStatus*>(ctx->host_status);
  const bool ok = rc == TREELSTM_OK;
  if (n_levels) *n_levels = ok ? hs->n_levels : 0;
  if (n_roots) *n_roots = ok ? (hs->n_roots < max_r ? hs->n_roots : max_r) : 0;
  ctx->launches = launches_fwd + (want_roots ? 1 : 0);
  return rc;
}

size_t treelstm_host_staging_bytes(const treelstm_t* ctx, int max_nodes) {
  if (!ctx || max_nodes < 0) return 0;
  return host_staging_layout(ctx, max_nodes < 1 ? 1 : (size_t)max_nodes).total;
}

int treelstm_set_host_staging(treelstm_t* ctx, void* device_buffer, size_t bytes) {
  if (!ctx) return TREELSTM_ERR_INVALID_ARG;
  if (device_buffer && reinterpret_cast<uintptr_t>(device_buffer) % 256 != 0) return TREELSTM_ERR_INVALID_ARG;
  free_host_path(ctx);
  ctx->hp.ext = static_cast<unsigned char*>(device_buffer);
  ctx->hp.ext_bytes = device_buffer ? bytes : 0;
  ctx->last.valid = false;
  return TREELSTM_OK;
}

int treelstm_selftest_waits(treelstm_t* ctx, void* workspace, size_t workspace_bytes, int32_t* result,
                            void* stream) {
  if (!ctx || !workspace || !result || workspace_bytes < sizeof(DevStatus)) return TREELSTM_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) % 256 != 0) return TREELSTM_ERR_INVALID_ARG;
  ctx->last.valid = false;   // the control block of an earlier forward may be the one overwritten
  ctx->last.ws = nullptr;    // and its workspace is no longer this context's to read
  return launch_selftest_waits(ctx, workspace, result, static_cast<cudaStream_t>(stream));
}

#ifdef TREELSTM_TRACE
// Trace builds only (not part of the public header): copies the cycle stamps of the last forward to
// the host, kTraceSlots per wavefront; which = 0 grid-wide kernel, 1 cluster kernel.  Synchronises.
TREELSTM_API int treelstm_trace_read(treelstm_t* ctx, int which, long long* out, int max_entries) {
  if (!ctx || !out || which < 0 || which > 2 || !ctx->last.ws) return TREELSTM_ERR_INVALID_ARG;
  if (which == 2) {   // the scheduler's phase stamps: the unused words of the control block
    DevStatus hs;
    TL_CUDA(ctx, cudaStreamSynchronize(ctx->last.stream));
    TL_CUDA(ctx, cudaMemcpy(&hs, static_cast<const char*>(ctx->last.ws) + ctx->last.lay.status, sizeof(hs), cudaMemcpyDeviceToHost));
    int cnt = 0;
    for (; cnt < 16 && cnt < max_entries; ++cnt) out[cnt] = hs.pad[cnt];
    return cnt;
  }
  const int total = kTraceSlots * kTraceLevels;
  const int cnt = max_entries < total ? max_entries : total;
  const char* src = static_cast<const char*>(ctx->last.ws) + ctx->last.lay.trace + (size_t)which * total * sizeof(long long);
  TL_CUDA(ctx, cudaStreamSynchronize(ctx->last.stream));
  TL_CUDA(ctx, cudaMemcpy(out, src, sizeof(long long) * cnt, cudaMemcpyDeviceToHost));
  return cnt;
}
#endif

int treelstm_last_launch_count(const treelstm_t* ctx) { return ctx ? ctx->launches : 0; }

int treelstm_last_mode(const treelstm_t* ctx) { return ctx && ctx->last.valid ? ctx->last.mode : -1; }

int treelstm_subforest_count(const treelstm_t* ctx) { return ctx && ctx->sf.ok ? ctx->sf.n_parts : 0; }

int treelstm_last_cuda_error(const treelstm_t* ctx) { return ctx ? ctx->cuda_error : 0; }

int treelstm_destroy(treelstm_t* ctx) {
  if (!ctx) return TREELSTM_OK;
  cudaFree(ctx->emb); cudaFree(ctx->W); cudaFree(ctx->b); cudaFree(ctx->Wc); cudaFree(ctx->bc); cudaFree(ctx->Wcat);
  cudaFree(ctx->emb_bf); cudaFree(ctx->Wp_h); cudaFree(ctx->Wp_x); cudaFree(ctx->bp_h); cudaFree(ctx->bp_x);
  if (ctx->host_level_offset) cudaFreeHost(ctx->host_level_offset);
  if (ctx->host_status) cudaFreeHost(ctx->host_status);
  free_host_path(ctx);
  if (ctx->ev_begin) cudaEventDestroy(ctx->ev_begin);
  if (ctx->ev_end) cudaEventDestroy(ctx->ev_end);
  delete ctx;
  return TREELSTM_OK;
}

const char* treelstm_strerror(int status) {
  switch (status) {
    case TREELSTM_OK: return "ok";
    case TREELSTM_ERR_INVALID_ARG: return "invalid argument";
    case TREELSTM_ERR_INVALID_FOREST: return "forest is not a set of disjoint binary trees";
    case TREELSTM_ERR_TOKEN_OUT_OF_RANGE: return "leaf token outside the vocabulary";
    case TREELSTM_ERR_LABEL_OUT_OF_RANGE: return "label outside the classifier's classes";
    case TREELSTM_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case TREELSTM_ERR_CUDA: return "CUDA runtime error";
    case TREELSTM_ERR_NO_DEVICE: return "no sm_100 CUDA device";
    case TREELSTM_ERR_UNSUPPORTED: return "size not supported";
    case TREELSTM_ERR_STATE: return "call order violated";
    case TREELSTM_ERR_CHECK: return "checked build: index out of range or state row written a wrong number of times";
    default: return "unknown status";
  }
}

}  // extern "C"
