// bf16 tensor-core wavefront evaluation (sm_100a: tcgen05.mma with the accumulator in tensor
// memory, both operands fetched by tiled TMA, cell update fused into the epilogue that drains
// tensor memory).
//
// Paper: Figure 2 (Section 3.1) - a node is LSTM(embed(word)) or LSTM(left_state, right_state);
// Section 2.2 - sibling subtrees are independent, so every node whose children are done can be
// evaluated at once.  Batching those nodes into one wide contraction is what Section 6.3 calls
// folding and charges with regrouping copies per depth; here nothing is regrouped between depths
// (see "No gather on the operand side" below).
//
// One tile = rt ready nodes (32, 64 or 128) x (8*G hidden units x 5 gates).  W is pre-packed so
// that the 5 gate pre-activations of a hidden unit sit in the same accumulator row slice and one
// thread (one tensor-memory lane = one node) can finish the cell without any exchange.
//
// No gather on the operand side: a tree node has exactly one caller, so the epilogue writes a
// node's state straight into the slot its caller will read - row pos(caller) of the dense operand
// matrix Ain[pos][h_l | h_r] (bf16) and of Cin[pos][c_l | c_r] (fp32), pos being the caller's
// position in the ready order.  Every wavefront's operand is then a contiguous block of rows, and
// one TMA request per operand brings a box of several (or all) K blocks of a tile.  Leaves: the
// embedding rows are copied once into ready order (Xin) by all CTAs before the first wavefront.
//
// Warp roles (384 threads): warps 0-3 and 6-9 epilogue (tensor-memory lane quadrant = warp id
// mod 4; the two sets split every unit group in halves), warp 4 TMA producer of the operand rows,
// warp 10 TMA producer of the weight rows (issuing a request costs its thread a few hundred
// cycles, so the two streams are issued side by side), warp 5 MMA issuer + tensor-memory owner,
// warp 11 chooses the tile plan of the next wavefront.
#include "tc_epilogue.cuh"

namespace tl {
namespace {

constexpr int kThreads = kTcThreads;
constexpr int kBBytes = kMaxG * kGColsI * 128;
constexpr int kRingBytes = kMaxStages * (kABytes + kGColsI * 128);   // 8 stages of the thinnest tile
constexpr int kCBytes = BM * 2 * kMaxG * 8 * 4;   // staged child cell states: 128 rows x 2 x 32 fp32
constexpr int kSmemBytes = kRingBytes + kCBytes + 1024 /*alignment slack*/ + 256 /*barriers*/ + 1024 /*row ids*/ +
                           4 * kLevelCache;
static_assert(kBBytes % 1024 == 0 && (kGColsI * 128) % 1024 == 0 && (kGColsL * 128) % 1024 == 0,
              "every TMA box lands on a 1024-byte boundary of the swizzle pattern");

// Tile shape of a wavefront: rt ready nodes (32, 64 or 128; the MMA always spans 128 rows, the rest
// of the accumulator is not stored) x g unit groups (1, 2 or 4).  Narrow wavefronts are cut into many
// small tiles (every SM gets one, each fetches little), wide ones into fat tiles (fewer re-reads of
// the operand rows).  Cost of a tile, fitted to clock64 traces and in units of 8 cycles: a fixed
// part (operand latency, tensor-memory hand-over, output copy) + rt (operand bytes) + 180 g (the
// epilogue's cell updates).  A wavefront that needs several rounds over the CTAs and whose last
// round has few tiles splits those into 2 or 4 column pieces (tail_ls), so that the last round costs
// a thin tile instead of a fat one.
// The operands of a tile arrive in boxes of kbox K blocks (one TMA request per operand and box); a
// box is one stage of the shared-memory ring: [kbox x rt operand rows | kbox x 40 g weight rows].
struct TilePlan {
  int g, lg, rt, lrt, tiles;
  int tail_from, tail_ls;                  // tiles from tail_from on are pieces of g >> tail_ls unit groups
  int sel, kbox, n_box, n_stages;          // sel 0: one box spans all K blocks, 1: boxes of two K blocks
  uint32_t a_bytes, w_bytes, stage_bytes;  // operand rows / weight rows (of a fat tile) of one K block; one stage
};
__host__ __device__ inline int tile_cost(int rt, int lg) { return 350 + rt + (180 << lg); }
__host__ __device__ inline TilePlan choose_tile_plan(int rows, int groups, int n_ctas, bool leaf, int kblocks) {
  TilePlan best{1, 0, BM, 7, 0, 0, 0, 0, 0, 0, 0, 0u, 0u, 0u};
  int best_cost = 1 << 30, best_rounds = 1;
  for (int lrt = 7; lrt >= (leaf ? 7 : 5); --lrt) {      // leaf rows come through a 128-row box only
    const int rt = 1 << lrt;
    const int mt = (rows + rt - 1) >> lrt;
    for (int lg = 0; lg <= 2; ++lg) {
      if (groups & ((1 << lg) - 1)) break;                // g must divide the number of unit groups
      const int fat = mt * (groups >> lg);
      int rounds = 1;
      while (rounds * n_ctas < fat) ++rounds;
      const int rem = fat - (rounds - 1) * n_ctas;        // tiles of the last round
      int ls = 0;
      if (rounds > 1) {
        ls = lg;
        while (ls > 0 && (rem << ls) > n_ctas) --ls;
      }
      const int cost = (rounds - 1) * tile_cost(rt, lg) + tile_cost(rt, lg - ls);
      if (cost < best_cost || (cost == best_cost && lg > best.lg)) {
        best_cost = cost;
        best_rounds = rounds;
        best.g = 1 << lg; best.lg = lg; best.rt = rt; best.lrt = lrt;
        best.tail_from = ls > 0 ? fat - rem : fat;
        best.tail_ls = ls;
        best.tiles = ls > 0 ? fat - rem + (rem << ls) : fat;
      }
    }
  }
  best.a_bytes = (uint32_t)best.rt * 128u;
  best.w_bytes = (uint32_t)(best.g * (leaf ? kGColsL : kGColsI)) * 128u;
  const uint32_t kb_bytes = best.a_bytes + best.w_bytes;
  // A wavefront done in one round takes each tile's operands in one request when they fit; with
  // several rounds, boxes of two K blocks let loads, MMAs and epilogues of consecutive tiles overlap.
  if (best_rounds == 1 && (uint32_t)kblocks * kb_bytes <= (uint32_t)kRingBytes) {
    best.sel = 0; best.kbox = kblocks; best.n_box = 1;
  } else {
    best.sel = 1; best.kbox = 2; best.n_box = (kblocks + 1) >> 1;
  }
  best.stage_bytes = (uint32_t)best.kbox * kb_bytes;
  best.n_stages = kMaxStages;
  while ((uint32_t)best.n_stages * best.stage_bytes > (uint32_t)kRingBytes) --best.n_stages;
  return best;
}

// ---- the kernel -------------------------------------------------------------------------------- //
// Before the first wavefront, spread over all threads of the grid:
//   * Xin[r] = emb_bf[token of the r-th leaf]: the embedding rows in ready order;
//   * slot[child] = 2 * pos + side for the two children of the node at every internal position pos
//     (where that child will deliver its state), slot[root] = -1.
__device__ void prepare_operands(const TcParams& p, int gtid, int gthreads) {
  const int n_leaves = p.level_offset[1];
  // the dependent loads of this thread's first slot entries and root go out before the gather, so
  // that the two chains of round trips run side by side
  const int pos0 = n_leaves + gtid;
  int l0 = -1, r0 = -1, root0 = -1;
  if (pos0 < p.n) {
    const int node = chk(p.st, p.order[pos0], p.n);
    l0 = chk(p.st, p.left[node], p.n);
    r0 = chk(p.st, p.right[node], p.n);
  }
  const int n_roots = p.st->n_roots;
  if (gtid < n_roots) root0 = chk(p.st, p.roots[gtid], p.n);
  gather_leaf_rows(p, 0, n_leaves, gtid >> 5, gthreads >> 5, gtid & 31);
  if (l0 >= 0) {
    p.slot[l0] = 2 * pos0;
    p.slot[r0] = 2 * pos0 + 1;
  }
  for (int pos = pos0 + gthreads; pos < p.n; pos += gthreads) {
    const int node = chk(p.st, p.order[pos], p.n);
    p.slot[chk(p.st, p.left[node], p.n)] = 2 * pos;
    p.slot[chk(p.st, p.right[node], p.n)] = 2 * pos + 1;
  }
  if (root0 >= 0) p.slot[root0] = -1;
  for (int t = gtid + gthreads; t < n_roots; t += gthreads) p.slot[chk(p.st, p.roots[t], p.n)] = -1;
}

// Leaves evaluated ahead of the schedule.  Their embedding rows: the same copy as gather_leaf_rows,
// for the rows [row_begin, row_end) of the kernel's own leaf order, with the token ids clamped into
// the vocabulary (nothing has been validated at that point).
__device__ __forceinline__ void gather_leaf_rows_unchecked(const TcParams& p, int row_begin, int row_end, int warp, int n_warps, int lane) {
  const int cpr = p.Ep / 8;                              // 16-byte chunks per row
  // a warp takes four rows at a time, all their loads in flight before the first store
  for (int base = row_begin + warp * 4; base < row_end; base += n_warps * 4) {
    const int my_row = base + (lane & 3);
    const int my_tok = my_row < row_end ? min(max(p.token[p.pre_order[my_row]], 0), p.vocab - 1) : 0;
    int tok[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) tok[k] = __shfl_sync(kFullMask, my_tok, k);
    for (int c0 = 0; c0 < cpr; c0 += 64) {
      uint4 v[4][2];
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int cc = c0 + h * 32 + lane;
          if (base + k < row_end && cc < cpr)
            v[k][h] = __ldg(reinterpret_cast<const uint4*>(p.emb_bf + (size_t)tok[k] * p.Ep) + cc);
        }
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int cc = c0 + h * 32 + lane;
          if (base + k < row_end && cc < cpr)
            reinterpret_cast<uint4*>(p.xin + (size_t)(base + k) * p.Ep)[cc] = v[k][h];
        }
    }
  }
}

// Once the schedule is known: every internal position pos (one warp each) gets the slots of its two
// children written - slot[child] = 2 * pos + side -, and a child that is a leaf has its state handed
// over right here: bf16 h (padded units as 0) and fp32 c into half `side` of the operand rows of pos.
// Roots get slot -1.
__device__ __forceinline__ void deliver_leaves(const TcParams& p, int gwarp, int n_warps, int lane) {
  const int H = p.H, Hp = p.Hp;
  const int n_leaves = p.level_offset[1];
  const bool vec = (H % 4) == 0;
  // A warp takes four positions at a time.  The chain of dependent loads (position -> node -> children
  // -> are they leaves) runs once for the four, every lane following position base + (lane & 3); then
  // the rows of a position's leaf children are loaded together before they are stored.
  for (int base = n_leaves + gwarp * 4; base < p.n; base += n_warps * 4) {
    const int pos = base + (lane & 3);
    int c0 = 0, c1 = 0, bits = 0;
    if (pos < p.n) {
      const int node = chk(p.st, p.order[pos], p.n);
      c0 = chk(p.st, p.left[node], p.n);
      c1 = chk(p.st, p.right[node], p.n);
      bits = (p.left[c0] < 0 ? 1 : 0) | (p.left[c1] < 0 ? 2 : 0);
      if (lane < 4) { p.slot[c0] = 2 * pos; p.slot[c1] = 2 * pos + 1; }
    }
    for (int k = 0; k < 4; ++k) {
      // the two children of position base + k; lane k holds their ids and whether they are leaves
      const int child0 = __shfl_sync(kFullMask, c0, k), child1 = __shfl_sync(kFullMask, c1, k);
      const int bb = __shfl_sync(kFullMask, bits, k);
      if (bb == 0) continue;
      const bool on0 = (bb & 1) != 0, on1 = (bb & 2) != 0;
      const float* hrow0 = p.h + (size_t)child0 * H;
      const float* crow0 = p.c + (size_t)child0 * H;
      const float* hrow1 = p.h + (size_t)child1 * H;
      const float* crow1 = p.c + (size_t)child1 * H;
      const size_t row = (size_t)(base + k) * 2;
      // two chunks of four units per lane and pass, all eight loads in flight before the stores
      for (int u0 = lane * 4; u0 < Hp; u0 += 256) {
        float hv[2][2][4], cv[2][2][4];   // [chunk][side][unit]
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int u = u0 + 128 * q;
#pragma unroll
          for (int sd = 0; sd < 2; ++sd) {
            const float* hrow = sd ? hrow1 : hrow0;
            const float* crow = sd ? crow1 : crow0;
            const bool on = sd ? on1 : on0;
            if (on && vec && u + 3 < H) {
              const float4 a = __ldcg(reinterpret_cast<const float4*>(hrow + u));
              const float4 b = __ldcg(reinterpret_cast<const float4*>(crow + u));
              hv[q][sd][0] = a.x; hv[q][sd][1] = a.y; hv[q][sd][2] = a.z; hv[q][sd][3] = a.w;
              cv[q][sd][0] = b.x; cv[q][sd][1] = b.y; cv[q][sd][2] = b.z; cv[q][sd][3] = b.w;
            } else {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const bool in = on && u + j < H;
                hv[q][sd][j] = in ? __ldcg(hrow + u + j) : 0.f;
                cv[q][sd][j] = in ? __ldcg(crow + u + j) : 0.f;
              }
            }
          }
        }
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const int u = u0 + 128 * q;
          if (u >= Hp) continue;
          const int count = min(4, H - u);
#pragma unroll
          for (int sd = 0; sd < 2; ++sd) {
            if (!(sd ? on1 : on0)) continue;
            __nv_bfloat162 lo = __floats2bfloat162_rn(hv[q][sd][0], hv[q][sd][1]), hi = __floats2bfloat162_rn(hv[q][sd][2], hv[q][sd][3]);
            *reinterpret_cast<uint2*>(p.ain + (row + sd) * Hp + u) =
                make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
            if (count > 0) st_row4(p.cin + (row + sd) * H + u, vec, count, cv[q][sd]);
          }
        }
      }
      if (lane == 0) {
        const int n_on = (on0 ? 1 : 0) + (on1 ? 1 : 0);
        count_write(p.chk_counts ? p.chk_counts + p.n : nullptr, base + k, n_on * H);
        count_write(p.chk_counts ? p.chk_counts + 2 * p.n : nullptr, base + k, n_on * H);
      }
    }
  }
  const int n_roots = p.st->n_roots;
  for (int t = gwarp * 32 + lane; t < n_roots; t += n_warps * 32) p.slot[chk(p.st, p.roots[t], p.n)] = -1;
}

__global__ void k_prepare_operands(TcParams p) {
  if (ld_volatile(&p.st->status) != 0) return;
  prepare_operands(p, blockIdx.x * blockDim.x + threadIdx.x, gridDim.x * blockDim.x);
}

// only_level >= 0: process that wavefront only (one launch per level; operands prepared before).
// only_level < 0: prepare the operands, then all wavefronts, separated by the bounded grid barrier (cooperative
// launch).
template <bool kLeavesFirst>
__global__ void __launch_bounds__(kThreads, 1)
k_fwd_tc(const __grid_constant__ TmapSet maps, TcParams p, int only_level) {
  // kLeavesFirst = false: the instantiation for launches that never take the leaves ahead of the schedule (one
  // launch per wavefront, cooperative launches); its code is the smaller one
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t tiles_addr = (raw_addr + 1023u) & ~1023u;
  unsigned char* tiles_ptr = smem_raw + (tiles_addr - raw_addr);
  const uint32_t cstage_addr = tiles_addr + kRingBytes;
  const unsigned char* cstage_ptr = tiles_ptr + kRingBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(tiles_ptr + kRingBytes + kCBytes);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty
  // bars[2S+4]: meeting point of the 256 epilogue threads (output staging)
  // bars[2S+5]: teardown after a failed wait - the MMA issuer's last commit
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 6);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  int* s_flag = const_cast<int*>(s_abort) + 1;
  int* s_rownode = reinterpret_cast<int*>(tiles_ptr + kRingBytes + kCBytes + 256);   // [128] node id of each tile row
  int* s_rowslot = s_rownode + BM;                                                   // [128] its delivery slot
  int* s_level_offset = s_rowslot + BM;   // first kLevelCache wavefront boundaries: no global round trip per level
  __shared__ TilePlan s_plan[2];          // tile plans of this and the next wavefront (written by warp 11)
  __shared__ unsigned int s_early;        // grid barrier: completion seen by the polling lane (see grid_barrier_with)
  __shared__ unsigned int s_pre;          // bit 0 / 1: first weight / operand box of the next wavefront requested ahead
  unsigned char* cstage_w = tiles_ptr + kRingBytes;
  const uint32_t epi_bar = smem_u32(bars + 2 * kMaxStages + 4);
  const uint32_t drain_bar = smem_u32(bars + 2 * kMaxStages + 5);
  uint32_t epi_phase = 0;
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 2 + a); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int Hp = p.Hp, H = p.H;
  const int groups = Hp / kUnitGroup;
  const int kb_leaf = p.Ep / kKBlock, kb_int = 2 * Hp / kKBlock;
  const bool vec = (H % 4) == 0;
  // Persistent mode with the leaves taken first (p.leaves_first): this kernel is launched as a
  // programmatic dependent of the ready-set construction and starts while that kernel still runs.
  // Leaves have no inputs to wait for (Section 4.1.1: an operation runs as soon as its inputs are
  // resolved), and their place in the ready order needs no dependency analysis - they are wavefront 0
  // in ascending node id.  So the CTAs rank the leaves themselves, fetch their embedding rows and
  // evaluate the whole leaf wavefront beside the scheduler; only then do they wait for it
  // (griddepcontrol.wait), and the leaves' states are handed to the callers' operand rows together
  // with the slot table, once the order of the internal nodes is known.
  constexpr bool leaves_first = kLeavesFirst;   // (the host launches that instantiation in persistent mode only, with p.leaves_first set)
#ifdef TREELSTM_TRACE
  long long* const trace = blockIdx.x == 0 && tid == 0 ? p.trace : nullptr;
  long long* const trace_cta = blockIdx.x == 0 ? p.trace : nullptr;   // stamps of the producers and the MMA issuer
#define TL_ROLE_STAMP(slot_first, slot_second)                                                        \
  do {                                                                                                \
    if (t < 2 * (int)gridDim.x) TL_STAMP(trace_cta, lvl, t < (int)gridDim.x ? (slot_first) : (slot_second)); \
  } while (0)
#else
#define TL_ROLE_STAMP(slot_first, slot_second) do { } while (0)
#endif
  // phases of a leaves-first run: the last row of the stamp table (slot 0: the kernel has started)
#define TL_PHASE_STAMP(slot) TL_STAMP(trace, kTraceLevels - 1, slot)
  TL_PHASE_STAMP(0);
  if (only_level < 0) {
    // Every CTA reads the packed weights and biases in every wavefront, but they may have left L2 since
    // the last call: all CTAs ask for a share of them now, and for the tensor maps, so that the first
    // tiles do not wait for memory.
    const int gtid = blockIdx.x * kThreads + tid, gthreads = gridDim.x * kThreads;
    warm_l2(p.wp_x, (size_t)groups * kGColsL * p.Ep * 2, gtid, gthreads);
    warm_l2(p.wp_h, (size_t)groups * kGColsI * 2 * Hp * 2, gtid, gthreads);
    warm_l2(p.bp_x, (size_t)groups * kGColsL * 4, gtid, gthreads);
    warm_l2(p.bp_h, (size_t)groups * kGColsI * 4, gtid, gthreads);
    if (tid < (int)(sizeof(TmapSet) / sizeof(CUtensorMap))) prefetch_tmap(reinterpret_cast<const CUtensorMap*>(&maps) + tid);
  }
  __shared__ int s_stop[2];
  __shared__ int s_scan[16];
  bool failed = false;
  int n_levels = 0, lvl_end = 0;
  // What the scheduler leaves behind is read here and nowhere before: its status, the number of
  // wavefronts, their boundaries, and where the grid-wide kernel stops (the narrow wavefronts at the end
  // of a forest may go to one cluster, launched next on the stream; without that launch the decision
  // is still worked out and left in the control block for the host to learn from).
  auto take_schedule = [&]() {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    failed = ld_volatile(&p.st->status) != 0;      // schedule failed: nothing to evaluate
    n_levels = failed ? 0 : p.st->n_levels;
    const int tail_from = only_level < 0 ? tail_first_level(p.level_offset, n_levels, p.tail_width, p.tail_min_levels, s_stop) : n_levels;
    if (only_level < 0 && !failed && blockIdx.x == 0 && tid == 0) p.st->tail_from = tail_from;
    lvl_end = only_level >= 0 ? only_level + 1 : (p.tail_launched ? tail_from : n_levels);
    for (int i = tid; i < kLevelCache && i <= n_levels; i += kThreads) s_level_offset[i] = p.level_offset[i];
  };
  if (!leaves_first) take_schedule();

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 256); }
    mbar_init(epi_bar, 256);
    mbar_init(drain_bar, 1);
    *s_abort = 0;
    s_early = 0u;
    s_pre = 0u;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(s_tmem), 512);   // columns: 2 accumulator stages x 256
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  // Pipeline positions; every role walks the same tile sequence, so they stay in step.  The ring
  // is re-cut at every wavefront (thin tiles leave room for more stages); each mbarrier keeps its
  // own phase, tracked per stage in a bit mask.
  uint32_t stage = 0, phase_bits = 0;   // smem ring (producer and MMA)
  uint32_t acc_iter = 0;                // accumulator ring (MMA and epilogue)
  uint32_t arrivals = 0;                // arrivals at the grid barrier expected so far
  bool alive = true;
  bool stop = false;                    // uniform over the CTA
  bool pre = false;                     // producers: this warp's first box of the wavefront was requested at the barrier
  uint32_t armed = 0;                   // producers (lane 0): ring stages this thread has requested a box into

  if (leaves_first) {
    // ---- the leaves' ranks: CTA b looks at the node ids [b * chunk, (b + 1) * chunk) ----
    // (the control block was cleared by the scheduler before it let this kernel start; its barrier
    // counter is this kernel's alone)
    const int chunk = (p.n + (int)gridDim.x - 1) / (int)gridDim.x;
    const int lo = min(p.n, (int)blockIdx.x * chunk), hi = min(p.n, lo + chunk);
    const int per = (hi - lo + kThreads - 1) / kThreads;
    const int my_lo = min(hi, lo + tid * per), my_hi = min(hi, my_lo + per);
    int mine = 0;
    for (int k = my_lo; k < my_hi; ++k)
      if (p.left[k] < 0) {
        ++mine;
        // the leaf's embedding row is wanted in L2 by the time the rows are copied into ready order
        const int tok = min(max(p.token[k], 0), p.vocab - 1);
        warm_l2(p.emb_bf + (size_t)tok * p.Ep, (size_t)p.Ep * 2, 0, 1);
      }
    // exclusive prefix over the threads of the CTA (and the total) of one int per thread
    auto cta_scan = [&](int v, int& total) {
      int inc = v;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_up_sync(kFullMask, inc, d);
        if (lane >= d) inc += o;
      }
      __syncthreads();
      if (lane == 31) s_scan[warp] = inc;
      __syncthreads();
      int before = 0, all = 0;
#pragma unroll
      for (int w2 = 0; w2 < kThreads / 32; ++w2) {
        const int c2 = s_scan[w2];
        if (w2 < warp) before += c2;
        all += c2;
      }
      total = all;
      return before + inc - v;
    };
    int cta_leaves = 0;
    TL_PHASE_STAMP(1);   // tensor memory and barriers set up, own share of the child array read
    const int my_first = cta_scan(mine, cta_leaves);
    if (tid == 0) p.pre_counts[blockIdx.x] = cta_leaves;
    arrivals += gridDim.x;
    if (!grid_barrier(p.st, arrivals, p.wait_limit, s_flag)) stop = true;
    TL_PHASE_STAMP(2);   // every CTA's leaf count is known
    int n_leaves = 0, base = 0;
    {
      // leaves in front of this CTA's node ids, and all of them (the grid has at most kThreads CTAs)
      const int v = tid < (int)gridDim.x ? __ldcg(p.pre_counts + tid) : 0;
      const int before = cta_scan(v, n_leaves);
      if (tid == (int)blockIdx.x) s_stop[0] = before;
      __syncthreads();
      base = s_stop[0];
    }
    if (!stop) {
      int rank = base + my_first;
      for (int k = my_lo; k < my_hi; ++k)
        if (p.left[k] < 0) p.pre_order[rank++] = k;
      __syncthreads();
      // the embedding rows of this CTA's leaves, in ready order (token ids are clamped: nothing has
      // been validated yet, and a forest the scheduler rejects must not make this kernel read astray)
      gather_leaf_rows_unchecked(p, base, base + cta_leaves, warp, kThreads / 32, lane);
      TL_PHASE_STAMP(3);   // own leaves ranked, their embedding rows copied
      asm volatile("fence.proxy.async.global;" ::: "memory");    // Xin is read through TMA
      arrivals += gridDim.x;
      if (!grid_barrier(p.st, arrivals, p.wait_limit, s_flag)) stop = true;
    }
    TL_PHASE_STAMP(4);   // all embedding rows are in place: the leaf wavefront starts
    if (tid == 0) { s_level_offset[0] = 0; s_level_offset[1] = n_leaves; }
    n_levels = n_leaves > 0 ? 1 : 0;
    lvl_end = n_levels;
    __syncthreads();
  } else if (only_level < 0 && n_levels > 0) {
    __syncthreads();                                            // the cached wavefront boundaries
    prepare_operands(p, blockIdx.x * kThreads + tid, gridDim.x * kThreads);
    asm volatile("fence.proxy.async.global;" ::: "memory");    // Xin is read through TMA
    arrivals += gridDim.x;
    if (!grid_barrier(p.st, arrivals, p.wait_limit, s_flag)) stop = true;
  }
  __syncthreads();

  const int lvl_begin = only_level >= 0 ? only_level : 0;
  auto level_begin = [&](int l) { return l < kLevelCache ? s_level_offset[l] : p.level_offset[l]; };
  auto make_plan = [&](int l) {
    return choose_tile_plan(level_begin(l + 1) - level_begin(l), groups, p.sched_ctas, l == 0, l == 0 ? kb_leaf : kb_int);
  };
  // Choosing a plan costs a few hundred cycles: one otherwise idle thread (warp 11) does it a
  // wavefront ahead, everybody else picks the result up after the barrier.
  if (warp == 11 && lane == 0 && lvl_begin < lvl_end) s_plan[lvl_begin & 1] = make_plan(lvl_begin);
  __syncthreads();
  // After the leaf wavefront of a leaves-first run: wait for the schedule, then every internal position
  // gets its slots written and the states of those of its children that are leaves.
  auto hand_leaves_over = [&]() {
    TL_PHASE_STAMP(5);   // all leaf states are in memory
    take_schedule();
    __syncthreads();
    TL_PHASE_STAMP(6);   // the scheduler has ended, its results are read
    if (n_levels > 0) {
      deliver_leaves(p, blockIdx.x * (kThreads / 32) + warp, gridDim.x * (kThreads / 32), lane);
      asm volatile("fence.proxy.async.global;" ::: "memory");    // the operand rows are read through TMA
    }
    if (warp == 11 && lane == 0 && 1 < lvl_end) s_plan[1] = make_plan(1);
    TL_PHASE_STAMP(7);   // slots written, leaf states handed to their callers
    arrivals += gridDim.x;
    if (!grid_barrier(p.st, arrivals, p.wait_limit, s_flag)) stop = true;
    TL_PHASE_STAMP(8);   // the first internal wavefront may start
  };
  if (leaves_first && (lvl_end == 0 || stop)) {
    // Nothing was evaluated: no leaf at all (the scheduler rejects such a forest) or a barrier gave
    // up.  The scheduler's status word is final once the wait has ended.
    take_schedule();
    if (!stop && !failed && tid == 0) report(p.st, TREELSTM_ERR_CHECK);   // a valid forest has leaves
    stop = true;
    lvl_end = 0;
  }
  for (int lvl = lvl_begin; lvl < lvl_end && !stop; ++lvl) {   // uniform trip count: barriers inside
    const int begin = level_begin(lvl), end = level_begin(lvl + 1);
    const bool leaf = lvl == 0;
    const TilePlan plan = s_plan[lvl & 1];
    TL_STAMP(trace, lvl, 0);
    if (warp == 11 && lane == 0 && lvl + 1 < lvl_end) s_plan[(lvl + 1) & 1] = make_plan(lvl + 1);
    const int rt = plan.rt;
    const int ntn = groups >> plan.lg;               // fat column tiles per row tile
    const int tiles = plan.tiles;
    const int kblocks = leaf ? kb_leaf : kb_int;
    const int gcols = leaf ? kGColsL : kGColsI;
    // A stage holds one box: kbox x rt operand rows, then kbox x ncols weight rows.  The MMA reads 128
    // rows from the start of a K block; what lies behind the rt fetched rows feeds accumulator rows
    // that are not stored.
    const uint32_t a_bytes = plan.a_bytes, stage_bytes = plan.stage_bytes;
    const uint32_t n_stages = (uint32_t)plan.n_stages;
    const int kbox = plan.kbox, n_box = plan.n_box;
    stage = 0;
    int nx_node = 0, nx_slot = -1;                  // epilogue: row data of this CTA's next tile, fetched a tile ahead
    bool nx_have = false;
    // leaves evaluated ahead of the schedule: their order is this kernel's own, and their states are
    // handed to the callers later (hand_leaves_over)
    const bool ahead = leaves_first && leaf;
    const int* const order_cur = ahead ? p.pre_order : p.order;

    for (int t = blockIdx.x; t < tiles && alive; t += gridDim.x) {
      // fat tile t = (row tile, column tile); a piece of the split last round is a column piece of a fat tile
      int lg = plan.lg, fat = t, piece = 0;
      if (t >= plan.tail_from) {
        const int u = t - plan.tail_from;
        fat = plan.tail_from + (u >> plan.tail_ls);
        piece = u & ((1 << plan.tail_ls) - 1);
        lg -= plan.tail_ls;
      }
      const int rtile = fat / ntn;
      const int nt = ((fat - rtile * ntn) << (plan.lg - lg)) + piece;   // column tile in units of G groups
      const int G = 1 << lg;
      const int ncols = G * gcols;                     // accumulator columns in use
      const int ncols_mma = (ncols + 15) & ~15;        // UMMA N (columns past ncols are never read)
      const uint32_t w_bytes = (uint32_t)ncols * 128u; // weight rows of one K block
      const int row0 = begin + (rtile << plan.lrt);
      const int row_end = min(end, row0 + rt);        // rows of this tile: [row0, row_end)

      if (warp == 4 || warp == 10) {
        // ---------------- operand producers (TMA) ----------------
        // Warp 4: the operand rows [row0, row0 + rt) of the dense operand matrix (rows past its end
        // read as zero; rows past the wavefront belong to later wavefronts and only feed accumulator
        // rows that are never stored).  Warp 10: the g unit groups of the packed weights.  One request
        // per box and operand; the two warps issue side by side.
        if (lane == 0) {
          const bool is_a = warp == 4;
          const CUtensorMap* map = is_a ? (leaf ? &maps.x[plan.sel] : &maps.a[plan.lrt - 5][plan.sel])
                                        : (leaf ? &maps.wx[lg][plan.sel] : &maps.wh[lg][plan.sel]);
          const uint32_t bytes = (uint32_t)kbox * (is_a ? a_bytes : w_bytes);
          const uint32_t off = is_a ? 0u : (uint32_t)kbox * a_bytes;
          const int y = is_a ? row0 : nt * ncols;
          for (int box = 0; box < n_box; ++box) {
            if (pre) {   // requested at the grid barrier
              pre = false;
              atomicAnd(&s_pre, is_a ? ~2u : ~1u);
              phase_bits ^= 1u << stage;
              if (++stage == n_stages) stage = 0;
              continue;
            }
            if (!mbar_wait(empty_bar(stage), ((phase_bits >> stage) & 1u) ^ 1u, s_abort, p.wait_limit, p.st)) {
              alive = false;
              break;
            }
            mbar_arrive_expect_tx(full_bar(stage), bytes);
            tma_load_3d(tiles_addr + stage * stage_bytes + off, map, 0, y, box * kbox, full_bar(stage));
            if (box == 0 && is_a) TL_ROLE_STAMP(14, 11);
            if (box == n_box - 1 && is_a) TL_ROLE_STAMP(15, 12);
            armed |= 1u << stage;
            phase_bits ^= 1u << stage;
            if (++stage == n_stages) stage = 0;
          }
        }
        __syncwarp();
        stage = __shfl_sync(kFullMask, stage, 0);
        phase_bits = __shfl_sync(kFullMask, phase_bits, 0);
        alive = __shfl_sync(kFullMask, (int)alive, 0) != 0;
      } else if (warp == 5) {
        // ---------------- MMA issuer ----------------
        if (lane == 0) {
          const uint32_t acc = acc_iter & 1, acc_phase = (acc_iter >> 1) & 1;
          if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1, s_abort, p.wait_limit, p.st)) alive = false;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + acc * kAccCols;
          const uint32_t idesc = umma_idesc(ncols_mma);
          bool first = true;
          for (int box = 0; box < n_box && alive; ++box) {
            if (!mbar_wait(full_bar(stage), (phase_bits >> stage) & 1u, s_abort, p.wait_limit, p.st)) {
              alive = false;
              break;
            }
            tc_fence_after();
            if (box == 0) TL_ROLE_STAMP(4, 13);
            const uint32_t st_addr = tiles_addr + stage * stage_bytes;
            const int nkb = min(kbox, kblocks - box * kbox);
            for (int kbi = 0; kbi < nkb; ++kbi) {
              const uint64_t a_desc = umma_desc(st_addr + (uint32_t)kbi * a_bytes);
              const uint64_t b_desc = umma_desc(st_addr + (uint32_t)kbox * a_bytes + (uint32_t)kbi * w_bytes);
#pragma unroll
              for (int k = 0; k < kKBlock / 16; ++k)   // UMMA K = 16 bf16 = 32 bytes = 2 descriptor units
                umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, !(first && k == 0));
              first = false;
            }
            umma_commit(empty_bar(stage));             // frees the stage when these MMAs retire
            phase_bits ^= 1u << stage;
            if (++stage == n_stages) stage = 0;
          }
          if (alive) umma_commit(tfull_bar(acc));      // the accumulator is complete
          TL_ROLE_STAMP(5, 5);
        }
        ++acc_iter;
      } else if (warp != 11) {
        // ---------------- epilogue: drain tensor memory, finish the cell ----------------
        // Two sets of four warps; set e takes hidden units [4e, 4e + 4) of every unit group.  A
        // warp may only read the tensor-memory lanes of quadrant (warp id mod 4).
        const int e = warp < 4 ? 0 : 1;   // warps 0-3: set 0, warps 6-9: set 1
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const int row = row0 + r;
        const bool valid = row < row_end;
        int node, slot;                               // slot: 2 * pos(caller) + side, -1 for a root
        if (nx_have) {
          node = nx_node; slot = nx_slot;
        } else {
          node = valid ? chk(p.st, order_cur[row], p.n) : 0;
          slot = valid && !ahead ? chk_slot(p.st, p.slot[node], p.n) : -1;
        }
        // the same two dependent loads for this CTA's next tile go out now and land while this tile is computed
        const int t2 = t + (int)gridDim.x;
        nx_have = t2 < tiles;
        bool valid2 = false;
        if (nx_have) {
          const int fat2 = t2 < plan.tail_from ? t2 : plan.tail_from + ((t2 - plan.tail_from) >> plan.tail_ls);
          const int rtile2 = fat2 / ntn, row2 = begin + (rtile2 << plan.lrt) + r;
          valid2 = r < rt && row2 < end;
          nx_node = valid2 ? chk(p.st, order_cur[row2], p.n) : 0;
        }
        EpiTile et;
        et.leaf = leaf; et.G = G; et.gcols = gcols; et.ncols = ncols; et.nt = nt;
        et.row = row; et.node = node; et.slot = slot; et.valid = valid;
        et.allow_staged_out = rt == BM;   // a tile of 32 or 64 rows writes so little that it stores straight from registers
        et.r = r; et.e = e; et.quad = quad;
        et.cstage_addr = cstage_addr; et.cstage_ptr = cstage_w; et.crow_shift = 8; et.half = 8;
        et.s_rownode = s_rownode; et.s_rowslot = s_rowslot;
        const uint32_t acc = acc_iter & 1;
        et.tmem_acc = tmem_base + acc * kAccCols;
        et.tfull = tfull_bar(acc); et.tempty = tempty_bar(acc); et.epi_bar = epi_bar; et.acc_phase = (acc_iter >> 1) & 1;
        et.bias = (leaf ? p.bp_x : p.bp_h) + nt * ncols + 4 * e;
#ifdef TREELSTM_TRACE
        // the CTA's first tile of the wavefront stamps slots 1-3, its second one slots 8-10
        if (trace != nullptr && lvl < kTraceLevels && t < 2 * (int)gridDim.x) et.stamp = trace + lvl * kTraceSlots + (t < (int)gridDim.x ? 1 : 8);
#endif
        epilogue_tile(p, et, epi_phase, alive, s_abort, [&]() { if (nx_have) nx_slot = valid2 && !ahead ? chk_slot(p.st, p.slot[nx_node], p.n) : -1; });
        ++acc_iter;
      }
    }
    // the operand rows the epilogue wrote are read through TMA (async proxy) by later wavefronts
    if (warp < 4 || (warp >= 6 && warp < 10)) asm volatile("fence.proxy.async.global;" ::: "memory");
    TL_STAMP(trace, lvl, 6);
    if (ahead) {
      // every CTA's leaf states must be in memory before anyone hands them on
      __syncthreads();
      if (*s_abort) break;
      arrivals += (uint32_t)min(tiles, (int)gridDim.x);
      if (!grid_barrier(p.st, arrivals, p.wait_limit, s_flag, (int)blockIdx.x < tiles)) break;
      hand_leaves_over();
      TL_STAMP(trace, lvl, 7);
      continue;
    }
    if (only_level < 0 && lvl + 1 < lvl_end) {
      // every role of every CTA joins the barrier.  A role that gave up has set s_abort before
      // this point, so the flag read after the CTA barrier is the same for all threads and the
      // loop is left by all of them together.
      __syncthreads();
      if (*s_abort) break;
      // only the CTAs that had a tile in this wavefront wrote anything: they arrive, the rest just wait
      arrivals += (uint32_t)min(tiles, (int)gridDim.x);
      // The first box of this CTA's first tile of the next wavefront is requested at the barrier, into
      // stage 0 of the re-cut ring (every MMA of this wavefront has retired: the epilogue waited for
      // them).  The weights do not depend on the wavefront before, so their producer asks at once;
      // the operand producer prepares its request and sends it the moment the polling lane reports
      // the barrier complete, ahead of the CTA-wide wake-up and the tile set-up.
      const uint32_t target = arrivals;
      const bool passed = grid_barrier_with(p.st, target, p.wait_limit, s_flag, (int)blockIdx.x < tiles, nullptr, &s_early, [&]() {
        if (lane != 0 || (warp != 4 && warp != 10)) return;
        const TilePlan np = s_plan[(lvl + 1) & 1];
        const int t = blockIdx.x;
        if (t >= np.tiles) return;
        int lg = np.lg, fat = t, piece = 0;
        if (t >= np.tail_from) {
          const int u = t - np.tail_from;
          fat = np.tail_from + (u >> np.tail_ls);
          piece = u & ((1 << np.tail_ls) - 1);
          lg -= np.tail_ls;
        }
        const int ntn2 = groups >> np.lg;
        const int rtile = fat / ntn2;
        if (!mbar_wait(empty_bar(0), (phase_bits & 1u) ^ 1u, s_abort, p.wait_limit, p.st)) return;
        if (warp == 10) {
          const int nt = ((fat - rtile * ntn2) << (np.lg - lg)) + piece;
          const int ncols = (1 << lg) * kGColsI;
          mbar_arrive_expect_tx(full_bar(0), (uint32_t)np.kbox * (uint32_t)ncols * 128u);
          tma_load_3d(tiles_addr + (uint32_t)np.kbox * np.a_bytes, &maps.wh[lg][np.sel], 0, nt * ncols, 0, full_bar(0));
          atomicOr(&s_pre, 1u);
          pre = true;
        } else {
          const int row0 = level_begin(lvl + 1) + (rtile << np.lrt);
          const CUtensorMap* map = &maps.a[np.lrt - 5][np.sel];
          const long long t0 = clock64();
          unsigned int seen;
          while ((seen = *(volatile unsigned int*)&s_early) != target) {
            if (seen == 0xFFFFFFFFu || clock64() - t0 > p.wait_limit) return;
          }
          __threadfence_block();
          mbar_arrive_expect_tx(full_bar(0), (uint32_t)np.kbox * np.a_bytes);
          tma_load_3d(tiles_addr, map, 0, row0, 0, full_bar(0));
          atomicOr(&s_pre, 2u);
          pre = true;
        }
      });
      if (!passed) break;
      TL_STAMP(trace, lvl, 7);
    }
  }

  // teardown: let in-flight asynchronous copies land before shared/tensor memory is released
  asm volatile("cp.async.wait_all;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (warp == 10 && lane == 0 && s_pre != 0u) {
    // the loop was left with a box requested ahead still in flight: stand in for the arrival of the
    // producer that did not ask, and let the data land
    if (s_pre != 3u) mbar_arrive(full_bar(0));
    mbar_drain(full_bar(0), phase_bits & 1u);
  }
  __syncthreads();
  if (*s_abort) {
    // A wait expired somewhere.  Before shared and tensor memory go back: every box a producer asked
    // for gets a bounded time to land (its barrier phase completes once both producers have arrived
    // and the bytes are in), and the MMAs issued so far a bounded time to retire.
    if ((warp == 4 || warp == 10) && lane == 0) {
      for (uint32_t s = 0; s < (uint32_t)kMaxStages; ++s)
        if (armed & (1u << s)) mbar_drain(full_bar(s), ((phase_bits >> s) & 1u) ^ 1u);
    }
    if (warp == 5 && lane == 0) {
      umma_commit(drain_bar);
      mbar_drain(drain_bar, 0);
    }
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// ---- self-test of the bounded waits ---------------------------------------------------------- //
// One CTA waits on an mbarrier nobody arrives at and on a grid barrier that expects a second CTA
// that does not exist.  Both waits must end by their cycle limit and record TREELSTM_ERR_TIMEOUT.
__global__ void k_selftest_waits(DevStatus* st, long long limit, int* result) {
  __shared__ uint64_t bar;
  __shared__ int s_abort, s_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  int outcome = 0;
  if (threadIdx.x == 0) {
    const bool ok = mbar_wait(smem_u32(&bar), 0, &s_abort, limit, st);
    outcome = ok ? 1 : 0;                 // 0 = gave up, as it must
  }
  const int after_mbar = ld_volatile(&st->status);
  if (threadIdx.x == 0) st->status = 0;   // second part starts clean
  __syncthreads();
  const bool ok2 = grid_barrier(st, 2u * gridDim.x, limit, &s_flag);
  if (threadIdx.x == 0) {
    result[0] = outcome;
    result[1] = after_mbar;
    result[2] = ok2 ? 1 : 0;
    result[3] = ld_volatile(&st->status);
  }
}

// ---- weight packing ---------------------------------------------------------------------------- //
// Packed row of hidden unit u, gate g (internal order i, f_l, f_r, o, u): (u/8)*40 + g*8 + u%8;
// leaf tiles keep gates i, o, u only: (u/8)*24 + gi*8 + u%8.  Each packed row holds the K vector.
__global__ void k_pack_weights(int H, int E, int Hp, int Ep, const float* W, const float* b,
                               __nv_bfloat16* Wp_h, __nv_bfloat16* Wp_x, float* bp_h, float* bp_x) {
  const int groups = Hp / 8;
  const size_t J = 5 * (size_t)H;
  const size_t total_h = (size_t)groups * 40 * 2 * Hp, total_x = (size_t)groups * 24 * Ep;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_h; i += stride) {
    const int k = (int)(i % (2 * Hp)), prow = (int)(i / (2 * Hp));
    const int u = (prow / 40) * 8 + prow % 8, g = (prow % 40) / 8;
    const int kk = k < Hp ? k : k - Hp;
    float v = 0.f;
    if (u < H && kk < H) v = W[(size_t)(E + (k < Hp ? 0 : H) + kk) * J + g * H + u];
    Wp_h[i] = __float2bfloat16_rn(v);
    if (k == 0) bp_h[prow] = u < H ? b[g * H + u] : 0.f;
  }
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total_x; i += stride) {
    const int k = (int)(i % Ep), prow = (int)(i / Ep);
    const int u = (prow / 24) * 8 + prow % 8, gi = (prow % 24) / 8;
    const int g = gi == 0 ? 0 : (gi == 1 ? 3 : 4);
    float v = 0.f;
    if (u < H && k < E) v = W[(size_t)k * J + g * H + u];
    Wp_x[i] = __float2bfloat16_rn(v);
    if (k == 0) bp_x[prow] = u < H ? b[g * H + u] : 0.f;
  }
}

__global__ void k_pack_embedding(int vocab, int E, int Ep, const float* emb, __nv_bfloat16* emb_bf) {
  const size_t total = (size_t)vocab * Ep, stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const int k = (int)(i % Ep);
    const size_t v = i / Ep;
    emb_bf[i] = __float2bfloat16_rn(k < E ? emb[v * E + k] : 0.f);
  }
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int make_tmap(treelstm* ctx, CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows,
              uint32_t box_kb) {
  static EncodeTiledFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    TL_CUDA(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
    if (!fn || q != cudaDriverEntryPointSuccess) return TREELSTM_ERR_CUDA;
    encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  // element (k, row, kb) of the view lives at base + kb * 128 + row * pitch + k * 2 bytes
  const cuuint64_t dims[3] = {kKBlock, rows, inner / kKBlock};
  const cuuint64_t strides[2] = {inner * 2, kKBlock * 2};   // bytes between rows, between K blocks
  const cuuint32_t box[3] = {kKBlock, box_rows, box_kb};    // 64 bf16 = one 128-byte swizzle span
  const cuuint32_t elem[3] = {1, 1, 1};
  CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, elem,
                      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) { ctx->cuda_error = (int)r; return TREELSTM_ERR_CUDA; }
  return TREELSTM_OK;
}

int ensure_operand_tmaps(treelstm* ctx, void* ws, int n, const void* xin, const void* ain) {
  if (ctx->tmap_ws_base == ws && ctx->tmap_ws_rows == n) return TREELSTM_OK;
  // the dense operands live in the caller's workspace
  const uint32_t kb_leaf = ctx->Ep / kKBlock, kb_int = 2 * ctx->Hp / kKBlock;
  for (int sel = 0; sel < 2; ++sel) {
    int rc = make_tmap(ctx, &ctx->maps.x[sel], xin, (uint64_t)ctx->Ep, (uint64_t)n, BM, sel == 0 ? kb_leaf : 2u);
    if (rc != TREELSTM_OK) return rc;
    for (int i = 0; i < 3; ++i) {
      rc = make_tmap(ctx, &ctx->maps.a[i][sel], ain, 2 * (uint64_t)ctx->Hp, (uint64_t)n, 32u << i,
                     sel == 0 ? kb_int : 2u);
      if (rc != TREELSTM_OK) return rc;
    }
  }
  ctx->tmap_ws_base = ws;
  ctx->tmap_ws_rows = n;
  return TREELSTM_OK;
}

int init_tc_attributes(treelstm* ctx) {
  TL_CUDA(ctx, cudaFuncSetAttribute(k_fwd_tc<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  TL_CUDA(ctx, cudaFuncSetAttribute(k_fwd_tc<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
  int per_sm = 0;
  TL_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fwd_tc<true>, kThreads, kSmemBytes));
  ctx->tc_resident_ctas = per_sm * ctx->sm_count;
  return TREELSTM_OK;
}

int launch_selftest_waits(treelstm* ctx, void* ws, int* result_dev, cudaStream_t stream) {
  DevStatus* st = static_cast<DevStatus*>(ws);
  TL_CUDA(ctx, cudaMemsetAsync(st, 0, sizeof(DevStatus), stream));
  k_selftest_waits<<<1, 64, 0, stream>>>(st, ctx->opt.wait_limit_kcycles * 1024, result_dev);
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

int pack_weights_bf16(treelstm* ctx, cudaStream_t stream) {
  k_pack_weights<<<512, 256, 0, stream>>>(ctx->H, ctx->E, ctx->Hp, ctx->Ep, ctx->W, ctx->b, ctx->Wp_h,
                                          ctx->Wp_x, ctx->bp_h, ctx->bp_x);
  k_pack_embedding<<<1024, 256, 0, stream>>>(ctx->vocab, ctx->E, ctx->Ep, ctx->emb, ctx->emb_bf);
  TL_CUDA(ctx, cudaGetLastError());
  const int groups = ctx->Hp / kUnitGroup;
  const uint32_t kb_leaf = ctx->Ep / kKBlock, kb_int = 2 * ctx->Hp / kKBlock;
  if (kb_leaf > 256 || kb_int > 256) return TREELSTM_ERR_UNSUPPORTED;   // a box dimension holds at most 256
  for (int sel = 0; sel < 2; ++sel)
    for (int lg = 0; lg < 3; ++lg) {
      // groups the number of unit groups does not divide into are never chosen; their maps stay valid anyway
      int rc = make_tmap(ctx, &ctx->maps.wh[lg][sel], ctx->Wp_h, 2 * (uint64_t)ctx->Hp, (uint64_t)groups * kGColsI,
                         (uint32_t)kGColsI << lg, sel == 0 ? kb_int : 2u);
      if (rc != TREELSTM_OK) return rc;
      rc = make_tmap(ctx, &ctx->maps.wx[lg][sel], ctx->Wp_x, (uint64_t)ctx->Ep, (uint64_t)groups * kGColsL,
                     (uint32_t)kGColsL << lg, sel == 0 ? kb_leaf : 2u);
      if (rc != TREELSTM_OK) return rc;
    }
  ctx->tmap_ws_base = nullptr;
  ctx->have_tmaps = true;
  return TREELSTM_OK;
}

int launch_forward_bf16(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                        const int32_t* token, float* h, float* c, const int32_t* order,
                        const int32_t* level_offset_dev, const int32_t* level_offset_host,
                        int n_levels_host, int flags, void* ws, const WsLayout& lay,
                        cudaStream_t stream) {
  if (!ctx->have_tmaps) return TREELSTM_ERR_STATE;
  char* base = static_cast<char*>(ws);
  TcParams p;
  p.n = n; p.H = ctx->H; p.Hp = ctx->Hp; p.Ep = ctx->Ep; p.sched_ctas = ctx->sm_count; p.vocab = ctx->vocab;
  p.chk_counts = check_counters(ws, lay);
  p.left = left; p.right = right; p.token = token;
  p.order = order;
  p.roots = reinterpret_cast<int*>(base + lay.roots);
  p.level_offset = level_offset_dev;
  p.emb_bf = ctx->emb_bf;
  p.slot = reinterpret_cast<int*>(base + lay.slot);
  p.xin = reinterpret_cast<__nv_bfloat16*>(base + lay.xin);
  p.ain = reinterpret_cast<__nv_bfloat16*>(base + lay.ain);
  p.cin = reinterpret_cast<float*>(base + lay.cin);
  p.bp_h = ctx->bp_h; p.bp_x = ctx->bp_x;
  p.wp_h = ctx->Wp_h; p.wp_x = ctx->Wp_x;
  p.h = h; p.c = c;
  p.gates = (flags & TREELSTM_SAVE_FOR_BACKWARD) ? reinterpret_cast<float*>(base + lay.gates) : nullptr;
  p.st = reinterpret_cast<DevStatus*>(base + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  p.level = nullptr; p.part_offset = nullptr; p.part_level_spill = nullptr; p.n_parts = 0; p.groups_per_cta = 0;
  // The narrow wavefronts at the end of a forest go to one cluster (tail_tc.cu) where that kernel
  // exists for these sizes; where the hand-over happens is decided on the device from the level table.
  // (the host only knows the node count: forests too large for a narrow tail to matter skip the second launch)
  const bool tail_possible = (flags & TREELSTM_PERSISTENT) && ctx->tail_ok && ctx->opt.tail_width > 0 &&
                             ctx->opt.max_ctas == 0 && n <= ctx->opt.tail_max_nodes && n >= 8;
  // the second launch costs a few microseconds even when the cluster finds nothing to do: it is left out
  // while the control block of the last forward that was read back says that there was no such tail
  const bool with_tail = tail_possible && !(ctx->tail_skip && ctx->opt.tail_min_levels == 0);
  p.tail_width = tail_possible ? ctx->opt.tail_width : 0;
  p.tail_min_levels = ctx->opt.tail_min_levels;
  p.tail_launched = with_tail ? 1 : 0;
  // Started under the single-CTA scheduler, the kernel takes the leaves first (the scratch of the
  // multi-CTA scheduler, unused then, holds its leaf order).
  const int single_max = ctx->opt.sched_single_cta_max < kSchedSingleMaxNodes ? ctx->opt.sched_single_cta_max : kSchedSingleMaxNodes;
  int grid_persistent = ctx->sm_count;                 // one CTA per SM (shared and tensor memory)
  if (ctx->opt.max_ctas > 0 && grid_persistent > ctx->opt.max_ctas) grid_persistent = ctx->opt.max_ctas;
  const bool overlap = (flags & TREELSTM_PERSISTENT) && ctx->opt.overlap_launch && n <= single_max &&
                       ctx->tc_resident_ctas >= ctx->sm_count && ctx->sm_count > 1 && ctx->sm_count <= kThreads;
  if (overlap && grid_persistent > ctx->sm_count - 1) grid_persistent = ctx->sm_count - 1;   // the scheduler keeps its SM
  p.leaves_first = overlap && n >= ctx->opt.leaves_first_min_nodes ? 1 : 0;
  p.pre_counts = reinterpret_cast<int*>(base + lay.pre);
  p.pre_order = reinterpret_cast<int*>(base + lay.pending);
  if (overlap) p.sched_ctas = ctx->sm_count - 1;   // the tile plans count on the CTAs that run
  p.trace = nullptr;
#ifdef TREELSTM_TRACE
  p.trace = reinterpret_cast<long long*>(base + lay.trace);
  // (a run started under the scheduler keeps the stamps of the run before: a clearing operation between
  // the two kernels would hold this one back until the scheduler has ended)
  if (!overlap) TL_CUDA(ctx, cudaMemsetAsync(p.trace, 0, sizeof(long long) * kTraceSlots * kTraceLevels, stream));
#endif
  {
    int rc = ensure_operand_tmaps(ctx, ws, n, p.xin, p.ain);
    if (rc != TREELSTM_OK) return rc;
  }

  const int groups = ctx->Hp / kUnitGroup;
  if (flags & TREELSTM_PERSISTENT) {
    int grid = grid_persistent;
    const int want = ((n + 31) / 32 + 1) * groups;       // never more CTAs than the thinnest tiling has tiles
    if (grid > want) grid = want;
    int only = -1;
    // The grid barrier needs every CTA resident.  Two ways to launch:
    //  * as a programmatic dependent of the kernel before it on the stream - the ready-set construction:
    //    the CTAs come up and do their set-up while that kernel still runs (it gives the go-ahead at its
    //    start) and wait for its results at griddepcontrol.wait.  The runtime takes this attribute on a
    //    plain launch only (measured: together with the cooperative attribute it has no effect), so
    //    residency rests on the grid being no larger than what the device holds at once (checked
    //    here) and on the device not being shared with other work; if CTAs cannot come up, the bounded
    //    barrier ends the kernel with TREELSTM_ERR_TIMEOUT.
    //  * as a cooperative launch (TREELSTM_OPT_OVERLAP_LAUNCH = 0): the runtime guarantees residency,
    //    and the kernel starts when the one before it has ended.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = kSmemBytes; cfg.stream = stream;
    cudaLaunchAttribute attr;
    if (overlap) {
      attr.id = cudaLaunchAttributeProgrammaticStreamSerialization; attr.val.programmaticStreamSerializationAllowed = 1;
    } else {
      attr.id = cudaLaunchAttributeCooperative; attr.val.cooperative = 1;
    }
    cfg.attrs = &attr; cfg.numAttrs = 1;
    if (p.leaves_first) TL_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_fwd_tc<true>, ctx->maps, p, only));
    else TL_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_fwd_tc<false>, ctx->maps, p, only));
    ctx->launches += 1;
    if (with_tail)
      return launch_forward_bf16_tail(ctx, n, left, right, token, h, c, order, level_offset_dev, flags, ws, lay, stream);
    return TREELSTM_OK;
  }
  if (n_levels_host > 0) {
    const int n_leaves = level_offset_host[1];
    const int blocks = (int)(((long long)n_leaves * (ctx->Ep / 8) + 255) / 256);
    k_prepare_operands<<<blocks < 1 ? 1 : (blocks > 2048 ? 2048 : blocks), 256, 0, stream>>>(p);
    ctx->launches += 1;
  }
  for (int lvl = 0; lvl < n_levels_host; ++lvl) {
    const int w = level_offset_host[lvl + 1] - level_offset_host[lvl];
    if (w <= 0) continue;
    const int tiles = choose_tile_plan(w, groups, p.sched_ctas, lvl == 0,
                                       lvl == 0 ? ctx->Ep / kKBlock : 2 * ctx->Hp / kKBlock).tiles;
    k_fwd_tc<false><<<tiles, kThreads, kSmemBytes, stream>>>(ctx->maps, p, lvl);
    ctx->launches += 1;
  }
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

}  // namespace tl

// Host-side view of the tile plan the bf16 wavefront kernel chooses on the device (same function).
extern "C" int treelstm_tile_plan(int rows, int H, int E, int n_ctas, int leaf, int32_t* out) {
  using namespace tl;
  if (rows < 1 || H < 1 || E < 1 || n_ctas < 1 || !out) return TREELSTM_ERR_INVALID_ARG;
  const int Hp = round_up(H, kKBlock), Ep = round_up(E, kKBlock);
  const TilePlan pl = choose_tile_plan(rows, Hp / kUnitGroup, n_ctas, leaf != 0, leaf ? Ep / kKBlock : 2 * Hp / kKBlock);
  out[0] = pl.rt; out[1] = pl.g; out[2] = pl.tiles; out[3] = pl.tail_from; out[4] = pl.tail_ls;
  out[5] = pl.kbox; out[6] = pl.n_box; out[7] = pl.n_stages; out[8] = (int32_t)pl.stage_bytes; out[9] = kRingBytes;
  return TREELSTM_OK;
}

