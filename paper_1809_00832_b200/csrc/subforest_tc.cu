// bf16 tensor-core evaluation of sub-forests on thread-block clusters (sm_100a).
//
// Paper: Section 2.2 - the trees of a batch, like sibling subtrees, are independent of each other;
// Section 4.1.1 - a node is ready once its inputs are resolved.  The scheduler deals the trees of
// the forest out to as many sub-forests as clusters fit on the GPU.  One cluster evaluates one
// sub-forest wavefront by wavefront, on its own: the wait between two wavefronts is the hardware
// cluster barrier (a fraction of a microsecond) instead of a grid-wide barrier through global
// memory, and nothing ever waits for another sub-forest.
//
// Inside a cluster the recurrent weights are stationary: CTA r of the cluster owns the gate columns
// of hidden units [r * 8 * g, (r + 1) * 8 * g) (g unit groups per CTA) and keeps that slice of the
// packed W_h in shared memory for the whole kernel, so an internal wavefront only streams its
// operand rows.  Every CTA walks all row tiles of a wavefront of its sub-forest; a tile is 128 ready
// nodes x (8 * g hidden units x 5 gates), accumulated in tensor memory by tcgen05.mma and finished
// by the same fused cell epilogue as the grid-wide kernel (gemm_tc.cu): a node's bf16 h and fp32 c
// go straight into the operand row of its caller, rows being positions in the ready order of the
// sub-forest, so every wavefront's operand is a contiguous block of rows fetched by tiled TMA.
//
// Warp roles as in gemm_tc.cu (384 threads): warps 0-3 and 6-9 epilogue, warp 4 TMA producer of the
// operand rows, warp 10 TMA producer of the W_x tiles of the leaf wavefront (and of the resident
// W_h slice), warp 5 MMA issuer; warp 11 only joins the barriers.
#include "tc_epilogue.cuh"

namespace tl {
namespace {

constexpr int kThreads = kTcThreads;
constexpr int kSmemLimit = 232448;       // 227 KB of dynamic shared memory per CTA
constexpr int kFixedBytes = 1024 /*alignment slack*/ + 256 /*barriers*/ + 1024 /*row ids*/ + 4 * (kLevelCache + 1);

struct SfLayout {
  uint32_t wres_bytes, ring_bytes, cstage_bytes, crow_shift, total;
};

// Shared-memory plan of one CTA: resident W_h slice | operand ring | child-cell / output staging.
__host__ __device__ inline SfLayout sf_layout(int Hp, int gpc) {
  SfLayout L;
  L.wres_bytes = (uint32_t)(2 * Hp / kKBlock) * (uint32_t)gpc * kGColsI * 128u;
  L.crow_shift = gpc <= 2 ? 7u : 8u;                       // staging row: 2 x (8 * gpc) fp32, padded to 128 / 256 B
  L.cstage_bytes = (uint32_t)BM << L.crow_shift;
  const int stage_leaf = kABytes + gpc * kGColsL * 128;
  int avail = kSmemLimit - 1024 /*static shared memory*/ - kFixedBytes - (int)L.wres_bytes - (int)L.cstage_bytes;
  int ring = kMaxStages * stage_leaf;
  if (ring > avail) ring = avail;
  if (ring < 0) ring = 0;
  L.ring_bytes = (uint32_t)ring & ~1023u;
  L.total = L.wres_bytes + L.ring_bytes + L.cstage_bytes + kFixedBytes;
  return L;
}

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// Hardware barrier of the cluster; every thread of every CTA of the cluster takes part.  Release /
// acquire: what the cluster's threads wrote before it (global memory included) is visible after it.
__device__ __forceinline__ void cluster_sync_all() {
  __syncwarp();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __launch_bounds__(kThreads, 1)
k_fwd_tc_subforest(const __grid_constant__ TmapSet maps, const __grid_constant__ SfTmapSet sfm, TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const int G = p.groups_per_cta;
  const SfLayout L = sf_layout(p.Hp, G);
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t wres_addr = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (wres_addr - raw_addr);
  const uint32_t ring_addr = wres_addr + L.wres_bytes;
  const uint32_t cstage_addr = ring_addr + L.ring_bytes;
  unsigned char* cstage_ptr = base_ptr + L.wres_bytes + L.ring_bytes;
  unsigned char* fixed_ptr = cstage_ptr + L.cstage_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(fixed_ptr);
  // bars[0..S) full, [S..2S) empty, [2S..2S+2) tmem_full, [2S+2..2S+4) tmem_empty,
  // bars[2S+4]: meeting point of the 256 epilogue threads, bars[2S+5]: resident W_h slice has landed,
  // bars[2S+6]: teardown after a failed wait - the MMA issuer's last commit
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 2 * kMaxStages + 7);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  int* s_nlev = const_cast<int*>(s_abort) + 1;
  int* s_rownode = reinterpret_cast<int*>(fixed_ptr + 256);   // [128] node id of each tile row
  int* s_rowslot = s_rownode + BM;                            // [128] its delivery slot
  int* s_loff = s_rowslot + BM;                               // wavefront boundaries of this sub-forest
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
  auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
  auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 2 + a); };
  const uint32_t epi_bar = bar0 + 8u * (2 * kMaxStages + 4);
  const uint32_t wres_bar = bar0 + 8u * (2 * kMaxStages + 5);
  const uint32_t drain_bar = bar0 + 8u * (2 * kMaxStages + 6);
  uint32_t epi_phase = 0;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // A failed schedule leaves the level count at 0.  (The status word is not used for this test: a
  // sibling cluster may record a timeout in it at any moment, and the CTAs of one cluster have to
  // take the same decision or the ones that stay would wait at the cluster barrier forever.)
  const int n_levels_all = ld_volatile(&p.st->n_levels);
  if (n_levels_all <= 0) return;
  const int cs = (int)cluster_nctarank(), rank = (int)cluster_ctarank();
  const int part = blockIdx.x / cs;
  const int pbeg = p.part_offset[part];
  const int pend = p.part_offset[part + 1];
  if (pbeg >= pend) return;                         // empty sub-forest: the whole cluster leaves
#ifdef TREELSTM_TRACE
  long long* const trace = blockIdx.x == 0 ? p.trace : nullptr;
#endif

  if (tid == 0) {
    for (int s = 0; s < kMaxStages; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 256); }
    mbar_init(epi_bar, 256);
    mbar_init(wres_bar, 1);
    mbar_init(drain_bar, 1);
    *s_abort = 0;
    *s_nlev = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(smem_u32(s_tmem), 512);   // 2 accumulator stages x 256 columns
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;

  const int Hp = p.Hp, H = p.H;
  const int kb_leaf = p.Ep / kKBlock, kb_int = 2 * Hp / kKBlock;
  const bool vec = (H % 4) == 0;
  const int nt = rank;                               // this CTA's slice of the hidden units

  // The slice of the packed recurrent weights this CTA keeps, fetched by one request: K block kb of
  // its 40 G packed rows at wres + kb * G * 5120 bytes (rows of 128 bytes, 128-byte swizzle).
  if (warp == 10 && lane == 0) {
    mbar_arrive_expect_tx(wres_bar, L.wres_bytes);
    tma_load_3d(wres_addr, &sfm.wres, 0, nt * G * kGColsI, 0, wres_bar);
  }

  // Wavefront boundaries of the sub-forest: its nodes are sorted by level, the levels are 0 .. top
  // without gaps.  Every CTA builds the table for itself.
  int* spill = p.part_level_spill + pbeg + part;     // entries past the shared-memory table
  for (int q = pbeg + tid; q < pend; q += kThreads) {
    const int lv = p.level[chk(p.st, p.order[q], p.n)];
    const int lvp = q > pbeg ? p.level[chk(p.st, p.order[q - 1], p.n)] : -1;
    if (lv != lvp) { if (lv <= kLevelCache) s_loff[lv] = q; else spill[lv] = q; }
    if (q == pend - 1) {
      if (lv + 1 <= kLevelCache) s_loff[lv + 1] = pend; else spill[lv + 1] = pend;
      *s_nlev = lv + 1;
    }
  }
  __syncthreads();
  const int n_levels = *s_nlev;
  auto loff = [&](int l) { return l <= kLevelCache ? s_loff[l] : __ldcg(spill + l); };

  // Operands of the sub-forest, spread over the threads of the cluster: embedding rows of its
  // leaves in ready order (Xin), and for every internal position the slots its two children
  // deliver their state to (slot[] of a root stays -1, set by the scheduler).
  {
    const int gtid = rank * kThreads + tid, gthreads = cs * kThreads;
    const int lend = loff(1);
    gather_leaf_rows(p, pbeg, lend, gtid >> 5, gthreads >> 5, lane);
    for (int pos = lend + gtid; pos < pend; pos += gthreads) {
      const int node = chk(p.st, p.order[pos], p.n);
      p.slot[chk(p.st, p.left[node], p.n)] = 2 * pos;
      p.slot[chk(p.st, p.right[node], p.n)] = 2 * pos + 1;
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");    // Xin is read through TMA
  }
  cluster_sync_all();

  uint32_t stage = 0, phase_bits = 0;   // operand ring (producers and MMA issuers)
  uint32_t acc_iter = 0;                // accumulator ring (MMA issuers and epilogue)
  bool alive = true;
  bool stop = false;                    // uniform over the CTA
  bool wres_ready = false;
  uint32_t armed = 0;                   // producers (lane 0): ring stages this thread has requested a box into

  // How a wavefront is cut up.  Worked out a wavefront ahead (before the cluster barrier, while the
  // stores of the current one drain), so that the first operand request goes out the moment the
  // barrier opens.
  struct LevelCfg {
    int begin, end, tiles, lrt, sel, kbox, n_box;
    uint32_t a_bytes, w_bytes, stage_bytes, n_stages;
    bool leaf;
  };
  auto make_cfg = [&](int lvl) {
    LevelCfg c;
    c.begin = loff(lvl); c.end = loff(lvl + 1);
    c.leaf = lvl == 0;
    const int rows = c.end - c.begin;
    c.tiles = (rows + BM - 1) / BM;
    const int kblocks = c.leaf ? kb_leaf : kb_int;
    // A wavefront of at most 64 (32) nodes fetches only that many operand rows; the MMA still
    // spans 128 rows, what lies behind the fetched rows feeds accumulator rows that are not stored.
    c.lrt = c.leaf || rows > 64 ? 7 : (rows > 32 ? 6 : 5);
    c.a_bytes = 128u << c.lrt;                                                // operand rows of one K block
    c.w_bytes = c.leaf ? (uint32_t)(G * kGColsL) * 128u : 0u;                 // leaf: W_x rows ride along; W_h is resident
    // A stage of the ring holds one box: kbox K blocks of operand rows (+ kbox K blocks of W_x rows).
    // A single-tile wavefront takes its operands in one request when they fit, anything else in
    // boxes of two K blocks so that loads, MMAs and epilogues of consecutive tiles overlap.
    c.sel = c.tiles == 1 && (uint32_t)kblocks * (c.a_bytes + c.w_bytes) <= L.ring_bytes ? 0 : 1;
    c.kbox = c.sel == 0 ? kblocks : 2;
    c.n_box = c.sel == 0 ? 1 : (kblocks + 1) >> 1;
    c.stage_bytes = (uint32_t)c.kbox * (c.a_bytes + c.w_bytes);
    c.n_stages = kMaxStages;
    while (c.n_stages * c.stage_bytes > L.ring_bytes) --c.n_stages;
    return c;
  };
  LevelCfg next_cfg = make_cfg(0);

  for (int lvl = 0; lvl < n_levels; ++lvl) {   // same trip count in every CTA of the cluster
    if (!stop) {
      const LevelCfg cfg = next_cfg;
      const int begin = cfg.begin, end = cfg.end;
      const bool leaf = cfg.leaf;
      const int rows = end - begin;
#ifdef TREELSTM_TRACE
      if (tid == 0) TL_STAMP(trace, lvl, 0);
#endif
      const int tiles = cfg.tiles;
      const int kblocks = leaf ? kb_leaf : kb_int;
      const int gcols = leaf ? kGColsL : kGColsI;
      const int ncols = G * gcols;                     // accumulator columns in use
      const int ncols_mma = (ncols + 15) & ~15;        // UMMA N (columns past ncols are never read)
      const int lrt = cfg.lrt, sel = cfg.sel, kbox = cfg.kbox, n_box = cfg.n_box;
      const uint32_t a_bytes = cfg.a_bytes, w_bytes = cfg.w_bytes, stage_bytes = cfg.stage_bytes, n_stages = cfg.n_stages;
      stage = 0;
      int nx_node = 0, nx_slot = -1;                // epilogue: row data of the next tile, fetched a tile ahead
      bool nx_have = false;

      for (int t = 0; t < tiles && alive; ++t) {
        const int row0 = begin + t * BM;

        if (warp == 4 || (warp == 10 && leaf)) {
          // ---------------- operand producers (TMA): one request per box and operand ----------------
          if (lane == 0) {
            const bool is_a = warp == 4;
            const CUtensorMap* map = is_a ? (leaf ? &maps.x[sel] : &maps.a[lrt - 5][sel]) : &sfm.wx[sel];
            const uint32_t bytes = (uint32_t)kbox * (is_a ? a_bytes : w_bytes);
            const uint32_t off = is_a ? 0u : (uint32_t)kbox * a_bytes;
            const int y = is_a ? row0 : nt * ncols;
            for (int box = 0; box < n_box; ++box) {
              if (!mbar_wait(empty_bar(stage), ((phase_bits >> stage) & 1u) ^ 1u, s_abort, p.wait_limit, p.st)) {
                alive = false;
                break;
              }
              mbar_arrive_expect_tx(full_bar(stage), bytes);
              tma_load_3d(ring_addr + stage * stage_bytes + off, map, 0, y, box * kbox, full_bar(stage));
#ifdef TREELSTM_TRACE
              if (is_a && t == 0 && box == 0) TL_STAMP(trace, lvl, 1);
#endif
              armed |= 1u << stage;
              if (is_a && !leaf) mbar_arrive(full_bar(stage));   // stands in for the W producer: W_h is resident
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
            if (!leaf && !wres_ready) {
              if (!mbar_wait(wres_bar, 0, s_abort, p.wait_limit, p.st)) alive = false;
              wres_ready = true;
            }
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
#ifdef TREELSTM_TRACE
              if (t == 0 && box == 0) TL_STAMP(trace, lvl, 2);
#endif
              const uint32_t st_addr = ring_addr + stage * stage_bytes;
              const int nkb = min(kbox, kblocks - box * kbox);
              for (int kbi = 0; kbi < nkb; ++kbi) {
                const uint32_t b_addr = leaf ? st_addr + (uint32_t)kbox * a_bytes + (uint32_t)kbi * w_bytes
                                             : wres_addr + (uint32_t)(box * kbox + kbi) * (uint32_t)ncols * 128u;
                const uint64_t a_desc = umma_desc(st_addr + (uint32_t)kbi * a_bytes), b_desc = umma_desc(b_addr);
#pragma unroll
                for (int k = 0; k < kKBlock / 16; ++k)   // UMMA K = 16 bf16 = 32 bytes = 2 descriptor units
                  umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, !(first && k == 0));
                first = false;
              }
              umma_commit(empty_bar(stage));             // frees the ring stage when these MMAs retire
              phase_bits ^= 1u << stage;
              if (++stage == n_stages) stage = 0;
            }
            if (alive) umma_commit(tfull_bar(acc));      // the accumulator is complete
#ifdef TREELSTM_TRACE
            if (t == tiles - 1) TL_STAMP(trace, lvl, 3);
#endif
          }
          ++acc_iter;
        } else if (warp != 10 && warp != 11) {
          // ---------------- epilogue: drain tensor memory, finish the cell ----------------
          const int e = warp < 4 ? 0 : 1;   // warps 0-3: units [0,4) of every group, warps 6-9: [4,8)
          const int quad = warp & 3;        // tensor-memory lane quadrant this warp may read
          const int r = quad * 32 + lane;
          const int row = row0 + r;
          const bool valid = row < end;
          int node, slot;                               // slot: 2 * pos(caller) + side, -1 for a root
          if (nx_have) {
            node = nx_node; slot = nx_slot;
          } else {
            node = valid ? chk(p.st, p.order[row], p.n) : 0;
            slot = valid ? chk_slot(p.st, p.slot[node], p.n) : -1;
          }
          // the same two dependent loads for the next tile go out now and land while this tile is computed
          nx_have = t + 1 < tiles;
          const bool valid2 = nx_have && row + BM < end;
          if (nx_have) nx_node = valid2 ? chk(p.st, p.order[row + BM], p.n) : 0;
          EpiTile et;
          et.leaf = leaf; et.G = G; et.gcols = gcols; et.ncols = ncols; et.nt = nt;
          et.row = row; et.node = node; et.slot = slot; et.valid = valid;
          et.allow_staged_out = rows > 64;   // a narrow tile writes so little that it stores straight from registers
          et.r = r; et.e = e; et.quad = quad;
          et.cstage_addr = cstage_addr; et.cstage_ptr = cstage_ptr; et.crow_shift = L.crow_shift;
          et.half = 4 << (L.crow_shift - 7);
          et.s_rownode = s_rownode; et.s_rowslot = s_rowslot;
          const uint32_t acc = acc_iter & 1;
          et.tmem_acc = tmem_base + acc * kAccCols;
          et.tfull = tfull_bar(acc); et.tempty = tempty_bar(acc); et.epi_bar = epi_bar; et.acc_phase = (acc_iter >> 1) & 1;
          et.bias = (leaf ? p.bp_x : p.bp_h) + nt * ncols + 4 * e;
#ifdef TREELSTM_TRACE
          if (tid == 0 && t == 0) TL_STAMP(trace, lvl, 4);
#endif
          epilogue_tile(p, et, epi_phase, alive, s_abort, [&]() { if (nx_have) nx_slot = valid2 ? chk_slot(p.st, p.slot[nx_node], p.n) : -1; });
#ifdef TREELSTM_TRACE
          if (tid == 0 && t == tiles - 1) TL_STAMP(trace, lvl, 5);
#endif
          ++acc_iter;
        }
      }
      // the operand rows the epilogue wrote are read through TMA (async proxy) by later wavefronts
      if (warp < 4 || (warp >= 6 && warp < 10)) asm volatile("fence.proxy.async.global;" ::: "memory");
#ifdef TREELSTM_TRACE
      if (tid == 0) TL_STAMP(trace, lvl, 6);
#endif
    }
    if (lvl + 1 < n_levels) {
      next_cfg = make_cfg(lvl + 1);
      // Every thread of the cluster meets here.  A CTA in which a wait expired keeps coming to the
      // barriers (its peers must not wait for it forever) but does no more work.
      cluster_sync_all();
      if (*s_abort) stop = true;
#ifdef TREELSTM_TRACE
      if (tid == 0) TL_STAMP(trace, lvl, 7);
#endif
    }
  }

  // teardown: let in-flight asynchronous copies land before shared/tensor memory is released
  if (warp == 10 && lane == 0 && !wres_ready) {
    if (*s_abort) mbar_drain(wres_bar, 0); else mbar_wait(wres_bar, 0, s_abort, p.wait_limit, p.st);
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  if (*s_abort) {
    // as in the grid-wide kernel: requested boxes get a bounded time to land, issued MMAs to retire
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

}  // namespace

// How the sub-forest kernel would run for this context: cluster size, unit groups per CTA, bytes of
// dynamic shared memory, and how many clusters are resident at once (= number of sub-forests).
// ok = false if the hidden size does not fit the weight-stationary plan.
SubforestPlan subforest_plan(treelstm* ctx) {
  SubforestPlan pl{};
  if (ctx->precision != TREELSTM_BF16) return pl;
  const int groups = ctx->Hp / kUnitGroup;
  int cs = 0;
  if (groups % 16 == 0) cs = 16; else if (groups % 8 == 0) cs = 8; else return pl;
  const int gpc = groups / cs;
  if (gpc < 1 || gpc > 3) return pl;
  const SfLayout L = sf_layout(ctx->Hp, gpc);
  if (L.ring_bytes < 3u * (kABytes + gpc * kGColsL * 128)) return pl;   // fewer than 3 leaf stages: not worth it
  if (cudaFuncSetAttribute(k_fwd_tc_subforest, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)L.total) != cudaSuccess ||
      cudaFuncSetAttribute(k_fwd_tc_subforest, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess) {
    cudaGetLastError();
    return pl;
  }
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(cs); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = L.total;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&n_clusters, k_fwd_tc_subforest, &cfg) != cudaSuccess || n_clusters < 1) {
    cudaGetLastError();
    return pl;
  }
  const uint32_t kb_leaf = ctx->Ep / kKBlock, kb_int = 2 * ctx->Hp / kKBlock;
  if (make_tmap(ctx, &ctx->sf_maps.wres, ctx->Wp_h, 2 * (uint64_t)ctx->Hp, (uint64_t)groups * kGColsI,
                (uint32_t)(gpc * kGColsI), kb_int) != TREELSTM_OK ||
      make_tmap(ctx, &ctx->sf_maps.wx[0], ctx->Wp_x, (uint64_t)ctx->Ep, (uint64_t)groups * kGColsL,
                (uint32_t)(gpc * kGColsL), kb_leaf) != TREELSTM_OK ||
      make_tmap(ctx, &ctx->sf_maps.wx[1], ctx->Wp_x, (uint64_t)ctx->Ep, (uint64_t)groups * kGColsL,
                (uint32_t)(gpc * kGColsL), 2u) != TREELSTM_OK)
    return pl;
  pl.ok = true;
  pl.cluster_size = cs;
  pl.groups_per_cta = gpc;
  pl.smem_bytes = (int)L.total;
  pl.n_parts = n_clusters < kMaxParts ? n_clusters : kMaxParts;
  return pl;
}

int launch_forward_bf16_subforest(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                                  const int32_t* token, float* h, float* c, const int32_t* level, int flags,
                                  void* ws, const WsLayout& lay, cudaStream_t stream) {
  if (!ctx->have_tmaps || !ctx->sf.ok) return TREELSTM_ERR_STATE;
  char* base = static_cast<char*>(ws);
  TcParams p{};
  p.n = n; p.H = ctx->H; p.Hp = ctx->Hp; p.Ep = ctx->Ep; p.sched_ctas = ctx->sm_count; p.vocab = ctx->vocab;
  p.chk_counts = check_counters(ws, lay);
  p.left = left; p.right = right; p.token = token;
  p.order = reinterpret_cast<int*>(base + lay.part_order);   // rows are positions in this order
  p.roots = reinterpret_cast<int*>(base + lay.roots);
  p.level_offset = nullptr;
  p.tail_width = 0;
  p.tail_min_levels = 0;
  p.tail_launched = 0;
  p.trace = nullptr;
#ifdef TREELSTM_TRACE
  p.trace = reinterpret_cast<long long*>(base + lay.trace) + kTraceSlots * kTraceLevels;
  TL_CUDA(ctx, cudaMemsetAsync(p.trace, 0, sizeof(long long) * kTraceSlots * kTraceLevels, stream));
#endif
  p.emb_bf = ctx->emb_bf;
  p.slot = reinterpret_cast<int*>(base + lay.slot);
  p.xin = reinterpret_cast<__nv_bfloat16*>(base + lay.xin);
  p.ain = reinterpret_cast<__nv_bfloat16*>(base + lay.ain);
  p.cin = reinterpret_cast<float*>(base + lay.cin);
  p.bp_h = ctx->bp_h; p.bp_x = ctx->bp_x;
  p.h = h; p.c = c;
  p.gates = (flags & TREELSTM_SAVE_FOR_BACKWARD) ? reinterpret_cast<float*>(base + lay.gates) : nullptr;
  p.st = reinterpret_cast<DevStatus*>(base + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  p.level = level;
  p.part_offset = reinterpret_cast<int*>(base + lay.part_offset);
  p.part_level_spill = reinterpret_cast<int*>(base + lay.part_spill);
  p.n_parts = ctx->sf.n_parts;
  p.groups_per_cta = ctx->sf.groups_per_cta;
  int rc = ensure_operand_tmaps(ctx, ws, n, p.xin, p.ain);
  if (rc != TREELSTM_OK) return rc;

  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = ctx->sf.cluster_size; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(ctx->sf.n_parts * ctx->sf.cluster_size);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = ctx->sf.smem_bytes;
  cfg.stream = stream;
  cfg.attrs = at; cfg.numAttrs = 1;
  TL_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_fwd_tc_subforest, ctx->maps, ctx->sf_maps, p));
  ctx->launches += 1;
  return TREELSTM_OK;
}

}  // namespace tl
