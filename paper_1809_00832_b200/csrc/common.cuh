// Internal declarations shared by the translation units of libtreelstm_b200.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/treelstm.h"

namespace tl {

// Device-resident control block at the start of the caller's workspace.  Zeroed at the start
// of every forward call.
struct DevStatus {
  int status;            // 0 or the most negative treelstm_status any kernel reported
  int n_levels;          // number of wavefronts
  int n_roots;           // number of trees
  int max_level;         // scratch of the multi-CTA level assignment
  unsigned int barrier;  // arrival counter of the persistent kernels' grid barrier
  int n_touched;         // distinct leaf tokens (backward)
  unsigned int barrier_bwd;  // arrival counter of the one-launch backward pass (cleared by its launch)
  int tail_from;         // persistent bf16 forward: first wavefront the cluster kernel takes (or would take), n_levels if none
  int pad[56];
};
static_assert(sizeof(DevStatus) == 256, "control block is one 256-byte line group");

// Offsets (bytes) of the regions inside the workspace for a forest of up to n nodes.
struct WsLayout {
  size_t status, parent, pending, order_tmp, level_offset, roots, table, slot, part_order, part_offset,
      part_spill, xin, ain, cin, gates, dh, dc, dz, tok_slot, trace, check, pre, total;
};

// Cycle stamps of the wavefront kernels (builds with -DTREELSTM_TRACE only): kTraceSlots stamps per
// wavefront for the first kTraceLevels wavefronts, written by the first CTA of each kernel.
constexpr int kTraceSlots = 16;
constexpr int kTraceLevels = 256;
#ifdef TREELSTM_TRACE
#define TL_STAMP(buf, level, slot)                                                            \
  do {                                                                                        \
    if ((buf) != nullptr && (level) < tl::kTraceLevels) (buf)[(level) * tl::kTraceSlots + (slot)] = clock64(); \
  } while (0)
#else
#define TL_STAMP(buf, level, slot) do { } while (0)
#endif

struct Options {
  int sched_single_cta_max = 32768;
  long long wait_limit_kcycles = 1 << 20;  // ~1e9 cycles, about half a second at 2 GHz
  int max_ctas = 0;
  int time_kernel = 0;
  int tail_width = 32;    // persistent bf16 forward: trailing wavefronts this narrow may run on one cluster (0: never)
  int tail_min_levels = 0; // > 0: hand them over if at least this many remain; 0: the device decides by its cost model
  int tail_max_nodes = 4096;   // forests with more nodes never launch the cluster kernel
  int leaves_first_min_nodes = 4096;   // forests at least this large: leaf wavefront before the wait for the schedule
  int dw_tensor_cores = 1;     // one-launch backward: dW and db by split-bf16 tensor-core contraction
  int overlap_launch = 1;      // persistent bf16 forward: the wavefront kernel starts under the scheduler (programmatic dependent launch)
};

constexpr int kRadixBins = 256;
constexpr int kRadixChunk = 1024;        // items per single-warp CTA of the multi-CTA sort
constexpr int kSchedSingleMaxNodes = 32768;
constexpr int kSchedPartMaxNodes = 24576;   // largest forest the single-CTA scheduler can also deal out to sub-forests
constexpr int kMaxParts = 32;               // upper bound on the number of sub-forests (co-resident clusters)

// Padded sizes of the tensor-core path: hidden units in groups of 8 (one packed weight group =
// 5 gates x 8 units = 40 rows), K blocks of 64 bf16 (one 128-byte swizzle span).
constexpr int kUnitGroup = 8;
constexpr int kKBlock = 64;

// Tiled tensor maps of the operands, all three-dimensional {64 elements (one 128-byte swizzle span),
// rows, K blocks} so that one request brings several K blocks of a tile.  Index [..][0]: the box
// spans all K blocks of the operand, [..][1]: two K blocks.
struct TmapSet {
  CUtensorMap a[3][2];    // operand rows of internal wavefronts (Ain), box rows 32 / 64 / 128
  CUtensorMap x[2];       // operand rows of the leaf wavefront (Xin), box rows 128
  CUtensorMap wh[3][2];   // packed recurrent weights, box rows 40 g for g = 1, 2, 4 unit groups
  CUtensorMap wx[3][2];   // packed input weights, box rows 24 g
};

// Maps of the sub-forest (cluster) kernel: its CTAs take g unit groups each, g = 1, 2 or 3.
struct SfTmapSet {
  CUtensorMap wres;       // packed recurrent weights, box = the whole slice of a CTA: 40 g rows x all K blocks
  CUtensorMap wx[2];      // packed input weights, box rows 24 g
};

// How the sub-forest (cluster) kernel runs for a context; ok = false: not available for its sizes.
struct SubforestPlan {
  bool ok = false;
  int cluster_size = 0, groups_per_cta = 0, smem_bytes = 0, n_parts = 0;
};

inline int round_up(int x, int m) { return (x + m - 1) / m * m; }
inline size_t round_up_sz(size_t x, size_t m) { return (x + m - 1) / m * m; }

}  // namespace tl

// The context behind the opaque handle of the C ABI.
struct treelstm {
  int H = 0, E = 0, vocab = 0, precision = 0, C = 0;
  int cell = 0;        // 0: TreeLSTM, else TREELSTM_CELL_TREERNN / TREELSTM_CELL_RNTN (no cell state, E == H)
  int Hp = 0, Ep = 0;  // bf16 path: H padded to a multiple of 64, E padded to a multiple of 64
  int device = 0;
  int sm_count = 0;

  // fp32 parameters (library-owned device copies)
  float* emb = nullptr;  // [vocab][E]
  float* W = nullptr;    // [E+2H][5H]
  float* b = nullptr;    // [5H]
  float* Wcat = nullptr; // TreeRNN / RNTN: [4H^2 + 2H][H] (tensor slices transposed, then W) or [2H][H]
  float* Wc = nullptr;   // [H][C]
  float* bc = nullptr;   // [C]

  // bf16 tensor-core path (library-owned)
  __nv_bfloat16* emb_bf = nullptr;  // [vocab][Ep]
  __nv_bfloat16* Wp_h = nullptr;    // [(Hp/8)*40][2*Hp]  packed recurrent weights, K contiguous
  __nv_bfloat16* Wp_x = nullptr;    // [(Hp/8)*24][Ep]    packed input weights (gates i, o, u)
  float* bp_h = nullptr;            // [(Hp/8)*40] bias in packed column order
  float* bp_x = nullptr;            // [(Hp/8)*24]
  tl::TmapSet maps;                     // passed to the kernels by value
  tl::SfTmapSet sf_maps;
  const void* tmap_ws_base = nullptr;   // the operand maps are rebuilt when the workspace or node count changes
  int tmap_ws_rows = 0;
  bool have_tmaps = false;
  tl::SubforestPlan sf;                 // filled at create (bf16 only)
  bool tail_ok = false;                 // the tail kernel exists for this context's sizes
  int tc_resident_ctas = 0;             // CTAs of the grid-wide bf16 kernel the device holds at once
  bool tail_skip = false;               // the last forward whose control block was read back had no tail worth a hand-over

  tl::Options opt;

  // what the last forward call saw (needed by roots / backward / status_sync)
  struct Last {
    bool valid = false;
    int n = 0, flags = 0, mode = 0;   // mode: which wavefront kernel ran (TREELSTM_PER_LEVEL / PERSISTENT / SUBFORESTS)
    const int32_t *left = nullptr, *right = nullptr, *token = nullptr;
    float *h = nullptr, *c = nullptr;
    int32_t *level = nullptr, *order = nullptr, *level_offset = nullptr;
    void* ws = nullptr;
    tl::WsLayout lay{};
    cudaStream_t stream = nullptr;
    bool host_levels_valid = false;
    int n_levels = 0;
  } last;
  int32_t* host_level_offset = nullptr;  // pinned, grows on demand
  int host_level_cap = 0;
  int* host_status = nullptr;            // pinned copy of DevStatus

  // buffers of treelstm_forward_host (library-owned, grown on demand)
  struct HostPath {
    int cap_nodes = 0;
    int32_t *forest = nullptr;       // [left | right | token] of the current call, packed
    unsigned char* roots_pack = nullptr;   // [root ids | root h | root c] of the current call, packed
    int32_t *left = nullptr, *right = nullptr, *token = nullptr, *level = nullptr, *order = nullptr,
            *n_levels = nullptr, *root_ids = nullptr, *n_roots = nullptr;   // left .. token, root_* point into the packs
    float *h = nullptr, *c = nullptr, *root_h = nullptr, *root_c = nullptr;
    void* ws = nullptr;
    size_t ws_bytes = 0;
    bool owned = false;              // the buffers above were allocated by the library (else carved from `ext`)
    unsigned char* ext = nullptr;    // caller-provided device staging memory (treelstm_set_host_staging)
    size_t ext_bytes = 0;
  } hp;

  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;  // around the wavefront kernel (optional)
  bool ev_valid = false;

  int launches = 0;
  int cuda_error = 0;
};

namespace tl {

WsLayout ws_layout(const treelstm* ctx, int n, bool with_backward);

// Per-device kernel attributes (the opt-in to more than 48 KB of dynamic shared memory belongs to the
// device that is current when it is set): called by treelstm_create with the context's device current.
int init_schedule_attributes(treelstm* ctx);   // schedule.cu
int init_tc_attributes(treelstm* ctx);         // gemm_tc.cu

// schedule.cu: enqueue the on-device ready-set construction.  Returns a treelstm_status.
int launch_schedule(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                    const int32_t* token, int32_t* level, int32_t* order, int32_t* level_offset,
                    int32_t* n_levels_out, void* ws, const WsLayout& lay, int n_parts, cudaStream_t stream);

// cell_fp32.cu
int launch_forward_fp32(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                        const int32_t* token, float* h, float* c, const int32_t* order,
                        const int32_t* level_offset_dev, const int32_t* level_offset_host,
                        int n_levels_host, int flags, void* ws, const WsLayout& lay,
                        cudaStream_t stream);

// cell_rec.cu (TreeRNN / RNTN)
int pack_weights_rec(treelstm* ctx, const float* W, const float* V, cudaStream_t stream);
int launch_forward_rec(treelstm* ctx, int n, const int32_t* left, const int32_t* right, const int32_t* token,
                       float* h, const int32_t* order, const int32_t* level_offset_dev,
                       const int32_t* level_offset_host, int n_levels_host, int flags, void* ws,
                       const WsLayout& lay, cudaStream_t stream);

// gemm_tc.cu
int pack_weights_bf16(treelstm* ctx, cudaStream_t stream);
int launch_forward_bf16(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                        const int32_t* token, float* h, float* c, const int32_t* order,
                        const int32_t* level_offset_dev, const int32_t* level_offset_host,
                        int n_levels_host, int flags, void* ws, const WsLayout& lay,
                        cudaStream_t stream);

// Rebuilds the tensor maps over the dense operands when the workspace or the node count changed.
int ensure_operand_tmaps(treelstm* ctx, void* ws, int n, const void* xin, const void* ain);

// subforest_tc.cu
SubforestPlan subforest_plan(treelstm* ctx);
int launch_forward_bf16_subforest(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                                  const int32_t* token, float* h, float* c, const int32_t* level, int flags,
                                  void* ws, const WsLayout& lay, cudaStream_t stream);

// tail_tc.cu: one cluster for the narrow wavefronts at the end of a forest
int init_tail_attributes(treelstm* ctx);
int launch_forward_bf16_tail(treelstm* ctx, int n, const int32_t* left, const int32_t* right, const int32_t* token,
                             float* h, float* c, const int32_t* order, const int32_t* level_offset_dev, int flags,
                             void* ws, const WsLayout& lay, cudaStream_t stream);

int launch_selftest_waits(treelstm* ctx, void* ws, int* result_dev, cudaStream_t stream);

// backward.cu
int launch_backward_rec(treelstm* ctx, const int32_t* labels, float* loss, float* dW, float* db, float* dV,
                        float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows, int32_t* n_touched,
                        cudaStream_t stream);
int ensure_host_levels(treelstm* ctx);
int launch_backward(treelstm* ctx, const int32_t* labels, float* loss, float* dW, float* db,
                    float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows,
                    int32_t* n_touched, cudaStream_t stream);

// dweight_tc.cu: dW += In^T dZ, db += sum dZ, dEmb_rows += dz_leaves W_x^T on the tensor cores (three bf16 pieces per fp32 value)
int init_dweight_tc_attributes(treelstm* ctx);
int launch_dweight_tc(treelstm* ctx, int n, const int32_t* order, const int32_t* level_offset, const int32_t* token,
                      const int32_t* left, const int32_t* right, const float* h, const float* dz, float* dW, float* db,
                      const int* tok_slot, float* dEmb_rows, DevStatus* st, cudaStream_t stream);

// Checked build: clears the per-row write counters before a forward / compares them after it
// (schedule.cu); both do nothing in the normal build.  Counters: [h per node | Ain per position | Cin per position].
int launch_check_clear(treelstm* ctx, int n, void* ws, const WsLayout& lay, cudaStream_t stream);
int launch_check_counts(treelstm* ctx, int n, const int32_t* rows, const int32_t* left, void* ws, const WsLayout& lay,
                        cudaStream_t stream);
inline int* check_counters(void* ws, const WsLayout& lay) {
#ifdef TREELSTM_CHECKED
  return reinterpret_cast<int*>(static_cast<char*>(ws) + lay.check);
#else
  (void)ws; (void)lay;
  return nullptr;
#endif
}

// roots (schedule.cu)
int launch_gather_roots(treelstm* ctx, int max_roots, int32_t* root_ids, float* root_h,
                        float* root_c, int32_t* n_roots, cudaStream_t stream);

#define TL_CUDA(ctx, expr)                                  \
  do {                                                      \
    cudaError_t e_ = (expr);                                \
    if (e_ != cudaSuccess) {                                \
      (ctx)->cuda_error = (int)e_;                          \
      return TREELSTM_ERR_CUDA;                             \
    }                                                       \
  } while (0)

#ifdef __CUDACC__
// Record an error in the control block; the most negative code wins.
__device__ __forceinline__ void report(DevStatus* st, int code) { atomicMin(&st->status, code); }

__device__ __forceinline__ int ld_volatile(const int* p) { return *(const volatile int*)p; }

// Checked build (-DTREELSTM_CHECKED; compute-sanitizer's stand-in where that tool is not available):
// every index that a kernel reads from the caller's arrays or from the schedule passes through
// chk() before it addresses anything - out of range: TREELSTM_ERR_CHECK is recorded and index 0 is
// used instead, so nothing is accessed out of bounds and nothing traps - and every store of state
// units is counted per row with count_write(); a kernel at the end of the forward compares the
// counts with what a correct evaluation writes (every node's h once, every internal position's
// operand row twice - one half per child).  In the normal build both compile to nothing.
#ifdef TREELSTM_CHECKED
__device__ __forceinline__ int chk(DevStatus* st, int idx, int limit) {
  if ((unsigned)idx < (unsigned)limit) return idx;
  report(st, TREELSTM_ERR_CHECK);
  return 0;
}
// delivery slots are 2 * position + side, or -1 for a root
__device__ __forceinline__ int chk_slot(DevStatus* st, int slot, int n) {
  if (slot == -1 || (unsigned)slot < 2u * (unsigned)n) return slot;
  report(st, TREELSTM_ERR_CHECK);
  return -1;
}
__device__ __forceinline__ void count_write(int* counter, int row, int units) {
  if (counter && units > 0) atomicAdd(counter + row, units);
}
#else
__device__ __forceinline__ int chk(DevStatus*, int idx, int) { return idx; }
__device__ __forceinline__ int chk_slot(DevStatus*, int slot, int) { return slot; }
__device__ __forceinline__ void count_write(int*, int, int) {}
#endif

// Bounded grid-wide barrier for cooperative (co-resident) launches.  `target` is the total
// number of arrivals expected so far (this barrier included).  A CTA that wrote nothing since the
// last barrier may pass arrive = false: it only waits, and the caller counts it out of `target`
// (arrivals on one counter are served one after the other, so fewer of them end the barrier sooner).
// Returns false if the wait expired or another CTA reported an error: the caller must then
// leave its level loop (every CTA sees the same outcome within one more barrier).
// The threads outside warp 0 run `while_waiting` between the arrival and the release.  A thread that
// wants to act the moment the barrier is complete, ahead of the CTA-wide wake-up, watches *s_early
// there: the polling lane that sees the last arrival stores `target` (unique per barrier) into it,
// 0xFFFFFFFF if the barrier failed.
template <class WaitFn>
__device__ __forceinline__ bool grid_barrier_with(DevStatus* st, unsigned int target,
                                                  long long limit_cycles, int* s_flag, bool arrive,
                                                  unsigned int* counter, unsigned int* s_early,
                                                  WaitFn while_waiting) {
  if (!counter) counter = &st->barrier;
  __syncthreads();
  if (threadIdx.x >= 32) while_waiting();
  if (threadIdx.x < 32) {
    // Warp 0 polls.  Lane 0 announces the arrival (release: everything this CTA wrote, ordered
    // before by the CTA barrier, is visible to whoever acquires the counter afterwards); then eight
    // lanes read the counter a fraction of a round trip apart, so that the last arrival is seen
    // after an eighth of the memory latency on average instead of half of it.
    if (threadIdx.x == 0) {
      *s_flag = -1;
      if (arrive) asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(counter) : "memory");
    }
    __syncwarp();
    const int lane = threadIdx.x;
    if (lane < 8) {
      const long long t0 = clock64();
      while (clock64() - t0 < 150 * lane) {}
      for (;;) {
        if (*(volatile int*)s_flag >= 0) break;          // another lane has the answer
        unsigned int seen;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
        if (seen >= target) {
          if (s_early) { __threadfence_block(); *(volatile unsigned int*)s_early = target; }
          *(volatile int*)s_flag = 1;
          break;
        }
        if (*(volatile int*)&st->status != 0) {
          if (s_early) *(volatile unsigned int*)s_early = 0xFFFFFFFFu;
          *(volatile int*)s_flag = 0;
          break;
        }
        if (clock64() - t0 > limit_cycles) {
          report(st, TREELSTM_ERR_TIMEOUT);
          if (s_early) *(volatile unsigned int*)s_early = 0xFFFFFFFFu;
          *(volatile int*)s_flag = 0;
          break;
        }
      }
    }
    __syncwarp();
  }
  __syncthreads();
  return *s_flag != 0;
}

__device__ __forceinline__ bool grid_barrier(DevStatus* st, unsigned int target,
                                             long long limit_cycles, int* s_flag, bool arrive = true,
                                             unsigned int* counter = nullptr) {
  return grid_barrier_with(st, target, limit_cycles, s_flag, arrive, counter, nullptr, []() {});
}
#endif

}  // namespace tl
