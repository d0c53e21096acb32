// dW = In^T dZ and db = sum dZ of the training step on the tensor cores, at fp32 accuracy.
//
// Paper, Section 4.2.2: the weight gradient of the recursive body sums one outer product
// in_n (x) dz_n per invocation n.  That sum is the only large contraction of a training step
// ((E + 2H) x 5H outputs, contraction over all nodes) and has no dependency between wavefronts, so
// it runs once, after the last wavefront, as a dense GEMM: tcgen05.mma with fp32 accumulators in
// tensor memory.  The fp32 path owes its callers fp32 results, and bf16 operands carry 8 mantissa
// bits, so every operand value v is split into three bf16 pieces v = v0 + v1 + v2 (v0 = bf16(v),
// v1 = bf16(v - v0), v2 = bf16(v - v0 - v1): together the 24 bits of v) and six products are
// accumulated: a0 b0 + a0 b1 + a1 b0 + a1 b1 + a0 b2 + a2 b0; the three that are left out are below
// 2^-24 of |a b|.
//
// Work item = (part, 128 input rows, 128 gate columns, a run of 64-node blocks).  part 0: the leaves,
// input rows = embedding units (In = embedding row of the leaf's token); part 1: the internal nodes,
// input rows = [h_l | h_r].  One more input row holds ones: its output row is db.  A CTA builds its
// operand tiles in shared memory itself, straight from the fp32 arrays (gathered through the
// schedule), in the layout the tensor core reads: K-major rows of 128 bytes, 128-byte swizzle - the
// node index is the contraction index, so this is a transposition, done on the fly: a thread takes one
// input row (or gate column) and eight consecutive nodes, which is one 16-byte piece of that layout.
// Two stages of tiles: block b + 1 is built while the MMAs of block b run.  Partial sums of the node
// runs meet in dW by atomic adds (dW and db are cleared before), whole rows at a time through a
// shared-memory copy of the accumulator.
#include "tc_ptx.cuh"

namespace tl {
namespace {

constexpr int kDwThreads = 256;
constexpr int kDwTile = 128;                     // rows of either operand tile (UMMA M and N)
constexpr int kDwBlock = 64;                     // nodes per block of the contraction (one swizzle span of bf16)
constexpr int kDwPieces = 3;                     // bf16 pieces per value
constexpr int kDwTileBytes = kDwTile * 128;      // one piece of one operand tile: 16 KB
constexpr int kDwStageBytes = 2 * kDwPieces * kDwTileBytes;   // A and B, three pieces each: 96 KB
constexpr int kDwStages = 2;
constexpr int kDwMaxRun = 8;                     // blocks per work item at most (index tables in shared memory)
constexpr int kDwSmemBytes = kDwStages * kDwStageBytes + 1024;   // + alignment slack

struct DwParams {
  int n, n_leaves, H, E, vocab;
  int run;                      // 64-node blocks per work item
  const int *order, *token, *left, *right;
  const int* level_offset;      // level_offset[1] = number of leaves (the host may not know it)
  const float *emb, *h, *dz, *W;
  const int* tok_slot;          // row of every token in dEmb_rows (third kind of work item only)
  float *dW, *db, *dEmb_rows;   // dEmb_rows == nullptr: the leaves' input gradients are not formed here
  DevStatus* st;
  long long wait_limit;
};

// (x, y) -> three words of two bf16 pieces each (x in the low half): x = x0 + x1 + x2, y likewise
__device__ __forceinline__ void split3_pair(float x, float y, uint32_t& w0, uint32_t& w1, uint32_t& w2) {
  auto pack = [](float a, float b) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&v);
  };
  w0 = pack(x, y);
  x -= __uint_as_float(w0 << 16);  y -= __uint_as_float(w0 & 0xFFFF0000u);
  w1 = pack(x, y);
  x -= __uint_as_float(w1 << 16);  y -= __uint_as_float(w1 & 0xFFFF0000u);
  w2 = pack(x, y);
}

// byte offset of the 16-byte piece (row r, nodes 8 c .. 8 c + 7) inside a K-major tile with the 128-byte swizzle
__device__ __forceinline__ uint32_t swz_piece(int r, int c) {
  return (uint32_t)((r >> 3) * 1024 + (r & 7) * 128 + ((c ^ (r & 7)) << 4));
}

// One operand tile (128 rows x 64 nodes, three pieces) of block `kb` of the work item, in two steps: the
// fp32 values into registers (tile_load: nothing but loads, so all of a block's are in flight together),
// then split, packed and stored into shared memory (tile_store).
// kKind 0: input rows of the leaves (embedding units, then the row of ones), 1: input rows of the internal
// nodes ([h_l | h_r], then the row of ones), 2: gate columns (dz).  row0: first row of the tile within its
// operand.  s_node / s_ia / s_ib: per node of the item its id and where its input row comes from (token; left,
// right child); entries behind the item's last node are 0 and their values are discarded.  Warp w takes the
// nodes 8 w .. 8 w + 7 of the block, lane l the rows l, l + 32, l + 64, l + 96.
template <int kKind>
__device__ __forceinline__ void tile_load(const DwParams& p, int row0, const int* s_node, const int* s_ia,
                                          const int* s_ib, int kb, float (&v)[4][8]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int H = p.H, E = p.E, J = 5 * H;
  const int rows = kKind == 0 ? E : (kKind == 1 ? 2 * H : J);
#pragma unroll
  for (int rg = 0; rg < 4; ++rg) {
    const int fc = min(row0 + rg * 32 + lane, rows - 1);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int k = kb * kDwBlock + 8 * warp + i;
      const float* src;
      if (kKind == 0) src = p.emb + (size_t)s_ia[k] * E + fc;
      else if (kKind == 1) src = p.h + (size_t)(fc < H ? s_ia[k] : s_ib[k]) * H + (fc < H ? fc : fc - H);
      else src = p.dz + (size_t)s_node[k] * J + fc;
      v[rg][i] = kKind == 0 ? __ldg(src) : *src;
    }
  }
}
template <int kKind>
__device__ __forceinline__ void tile_store(const DwParams& p, unsigned char* tile, int row0, int valid_nodes,
                                           const float (&v)[4][8]) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rows = kKind == 0 ? p.E : (kKind == 1 ? 2 * p.H : 5 * p.H);   // row `rows` of an input operand is the ones
#pragma unroll
  for (int rg = 0; rg < 4; ++rg) {
    const int r = rg * 32 + lane, f = row0 + r;
    uint32_t w0[4], w1[4], w2[4];
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
      float x[2];
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const bool node_ok = 8 * warp + i + e < valid_nodes;
        x[e] = node_ok && f < rows ? v[rg][i + e] : 0.f;
        if (kKind != 2 && node_ok && f == rows) x[e] = 1.f;
      }
      split3_pair(x[0], x[1], w0[i >> 1], w1[i >> 1], w2[i >> 1]);
    }
    unsigned char* dst = tile + swz_piece(r, warp);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w0[0], w0[1], w0[2], w0[3]);
    *reinterpret_cast<uint4*>(dst + kDwTileBytes) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
    *reinterpret_cast<uint4*>(dst + 2 * kDwTileBytes) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
  }
}

// The third kind of work item, dEmb_rows += dz_leaves W_x^T, contracts over the gate columns, which are
// contiguous in both operands (a leaf's dz row, a row of W): no transposition, a thread takes eight
// consecutive columns of one row - one 16-byte piece - for four rows.  row_ptr(r): start of tile row r in
// global memory or nullptr; j0: first column of the block; J: columns in a row.
template <class RowFn>
__device__ __forceinline__ void rows_load(RowFn row_ptr, int j0, int J, float (&v)[4][8]) {
  const int c = threadIdx.x & 7;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float* row = row_ptr((threadIdx.x >> 3) + 32 * i);
#pragma unroll
    for (int e = 0; e < 8; ++e) v[i][e] = row[min(j0 + 8 * c + e, J - 1)];
  }
}
__device__ __forceinline__ void rows_store(unsigned char* tile, int rows_valid, int j0, int J, const float (&v)[4][8]) {
  const int c = threadIdx.x & 7;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = (threadIdx.x >> 3) + 32 * i;
    uint32_t w0[4], w1[4], w2[4];
#pragma unroll
    for (int e = 0; e < 8; e += 2) {
      const float x = r < rows_valid && j0 + 8 * c + e < J ? v[i][e] : 0.f;
      const float y = r < rows_valid && j0 + 8 * c + e + 1 < J ? v[i][e + 1] : 0.f;
      split3_pair(x, y, w0[e >> 1], w1[e >> 1], w2[e >> 1]);
    }
    unsigned char* dst = tile + swz_piece(r, c);
    *reinterpret_cast<uint4*>(dst) = make_uint4(w0[0], w0[1], w0[2], w0[3]);
    *reinterpret_cast<uint4*>(dst + kDwTileBytes) = make_uint4(w1[0], w1[1], w1[2], w1[3]);
    *reinterpret_cast<uint4*>(dst + 2 * kDwTileBytes) = make_uint4(w2[0], w2[1], w2[2], w2[3]);
  }
}

struct DwShape {
  int rows[2], nodes[2], first_pos[2], m_tiles[2], runs[2], items[3], n_tiles;
  // third kind (input gradients of the leaves): tiles of 128 leaves x 128 embedding units, contraction over
  // the 64-column blocks of the gate columns that are not all forget gates (those are zero for a leaf)
  int leaf_tiles, e_tiles, kblocks, skip_first, skip_count, runs2;
};
__host__ __device__ inline DwShape dw_shape(int n, int n_leaves, int H, int E, int run, bool leaf_dinput) {
  DwShape s;
  s.rows[0] = E; s.rows[1] = 2 * H;
  s.nodes[0] = n_leaves; s.nodes[1] = n - n_leaves;
  s.first_pos[0] = 0; s.first_pos[1] = n_leaves;
  s.n_tiles = (5 * H + kDwTile - 1) / kDwTile;
  for (int q = 0; q < 2; ++q) {
    s.m_tiles[q] = (s.rows[q] + 1 + kDwTile - 1) / kDwTile;   // + 1: the row of ones
    const int blocks = (s.nodes[q] + kDwBlock - 1) / kDwBlock;
    s.runs[q] = (blocks + run - 1) / run;
    s.items[q] = s.m_tiles[q] * s.n_tiles * s.runs[q];
  }
  const int all = (5 * H + kDwBlock - 1) / kDwBlock;
  s.skip_first = (H + kDwBlock - 1) / kDwBlock;              // first block that starts inside [H, 3H)
  const int skip_end = 3 * H / kDwBlock;                     // first block that ends outside it
  s.skip_count = skip_end > s.skip_first ? skip_end - s.skip_first : 0;
  s.kblocks = all - s.skip_count;
  s.leaf_tiles = (n_leaves + kDwTile - 1) / kDwTile;
  s.e_tiles = (E + kDwTile - 1) / kDwTile;
  s.runs2 = (s.kblocks + run - 1) / run;
  s.items[2] = leaf_dinput ? s.leaf_tiles * s.e_tiles * s.runs2 : 0;
  return s;
}
// The number of 64-wide blocks per work item: as few as give every CTA of the grid at most one item.
__host__ __device__ inline int dw_run(int n, int n_leaves, int H, int E, bool leaf_dinput, int ctas) {
  int run = 1;
  for (; run < kDwMaxRun; ++run) {
    const DwShape s = dw_shape(n, n_leaves, H, E, run, leaf_dinput);
    if (s.items[0] + s.items[1] + s.items[2] <= ctas) break;
  }
  return run;
}

__global__ void __launch_bounds__(kDwThreads, 1) k_bwd_dweight_tc(DwParams p) {
  extern __shared__ unsigned char dw_dyn[];
  __shared__ int s_node[kDwMaxRun * kDwBlock], s_ia[kDwMaxRun * kDwBlock], s_ib[kDwMaxRun * kDwBlock];
  __shared__ __align__(8) uint64_t s_bars[kDwStages + 2];
  __shared__ uint32_t s_tmem;
  __shared__ int s_abort;
  if (ld_volatile(&p.st->status) != 0) return;   // the passes before failed: nothing here may be trusted
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  unsigned char* tiles = dw_dyn + ((1024u - (smem_u32(dw_dyn) & 1023u)) & 1023u);
  const uint32_t tiles_addr = smem_u32(tiles);
  const uint32_t stage_bar0 = smem_u32(&s_bars[0]), acc_bar = smem_u32(&s_bars[kDwStages]),
                 drain_bar = smem_u32(&s_bars[kDwStages + 1]);
  if (tid == 0) {
    for (int s = 0; s < kDwStages; ++s) mbar_init(stage_bar0 + 8 * s, 1);
    mbar_init(acc_bar, 1);
    mbar_init(drain_bar, 1);
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) tmem_alloc(smem_u32(&s_tmem), kDwTile);   // 128 columns: one 128 x 128 fp32 accumulator
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = s_tmem;
  const int H = p.H, E = p.E, J = 5 * H;
  const int n_leaves = p.st->n_levels > 0 ? min(p.n, max(0, p.level_offset[1])) : 0;
  const bool leaf_dinput = p.dEmb_rows != nullptr;
  const int run = dw_run(p.n, n_leaves, H, E, leaf_dinput, (int)gridDim.x);   // the host does not know the number of leaves
  const DwShape sh = dw_shape(p.n, n_leaves, H, E, run, leaf_dinput);
  const uint32_t idesc = umma_idesc(kDwTile);
  uint32_t built = 0, items_done = 0;   // blocks built / items finished by this CTA so far (barrier phases)
  bool failed = false;
  for (int item = blockIdx.x; item < sh.items[0] + sh.items[1] + sh.items[2] && !failed; item += gridDim.x) {
    const int part = item < sh.items[0] ? 0 : (item < sh.items[0] + sh.items[1] ? 1 : 2);
    int it = item - (part > 0 ? sh.items[0] : 0) - (part > 1 ? sh.items[1] : 0);
    int m0, j0, pos0 = 0, pos_end = 0, nblk, kb0 = 0, rows_here = 0;
    if (part < 2) {
      const int nt = it % sh.n_tiles; it /= sh.n_tiles;
      const int mt = it % sh.m_tiles[part], ri = it / sh.m_tiles[part];
      m0 = mt * kDwTile; j0 = nt * kDwTile;
      pos0 = sh.first_pos[part] + ri * run * kDwBlock;
      pos_end = min(sh.first_pos[part] + sh.nodes[part], pos0 + run * kDwBlock);
      nblk = (pos_end - pos0 + kDwBlock - 1) / kDwBlock;
      // the item's nodes and where their input rows come from
      for (int t = tid; t < nblk * kDwBlock; t += kDwThreads) {
        int node = 0, ia = 0, ib = 0;
        if (pos0 + t < pos_end) {
          node = chk(p.st, p.order[pos0 + t], p.n);
          if (part == 0) ia = chk(p.st, p.token[node], p.vocab);
          else { ia = chk(p.st, p.left[node], p.n); ib = chk(p.st, p.right[node], p.n); }
        }
        s_node[t] = node; s_ia[t] = ia; s_ib[t] = ib;
      }
    } else {
      const int et = it % sh.e_tiles; it /= sh.e_tiles;
      const int lt = it % sh.leaf_tiles, ri = it / sh.leaf_tiles;
      m0 = lt * kDwTile;                 // first leaf (position in the ready order: the leaves are wavefront 0)
      j0 = et * kDwTile;                 // first embedding unit
      rows_here = min(kDwTile, n_leaves - m0);
      kb0 = ri * run;                    // first of the item's blocks among those that are not skipped
      nblk = min(run, sh.kblocks - kb0);
      // the tile's leaves and their rows of dEmb_rows
      for (int t = tid; t < kDwTile; t += kDwThreads) {
        int node = 0, slot = 0;
        if (t < rows_here) {
          node = chk(p.st, p.order[m0 + t], p.n);
          slot = chk(p.st, p.tok_slot[chk(p.st, p.token[node], p.vocab)], n_leaves);
        }
        s_node[t] = node; s_ia[t] = slot;
      }
    }
    __syncthreads();
    for (int b = 0; b < nblk; ++b, ++built) {
      const uint32_t stage = built & 1u, use = built >> 1;
      unsigned char* st_tiles = tiles + stage * kDwStageBytes;
      const int valid_nodes = min(kDwBlock, pos_end - pos0 - b * kDwBlock);
      int kcol = 0;                      // part 2: first gate column of the block
      if (part == 2) {
        const int kb = kb0 + b;
        kcol = (kb < sh.skip_first ? kb : kb + sh.skip_count) * kDwBlock;
      }
      float va[4][8], vb[4][8];
      if (part == 0) tile_load<0>(p, m0, s_node, s_ia, s_ib, b, va);
      else if (part == 1) tile_load<1>(p, m0, s_node, s_ia, s_ib, b, va);
      else rows_load([&](int r) { return p.dz + (size_t)s_node[r] * J; }, kcol, J, va);
      if (part < 2) tile_load<2>(p, j0, s_node, s_ia, s_ib, b, vb);
      else rows_load([&](int r) { return p.W + (size_t)min(j0 + r, E - 1) * J; }, kcol, J, vb);
      bool ok = true;
      if (use >= 1)   // the MMAs that read this stage two blocks ago must have retired before it is overwritten
        ok = mbar_wait(stage_bar0 + 8 * stage, (use - 1) & 1u, &s_abort, p.wait_limit, p.st);
      if (__syncthreads_or(!ok)) { failed = true; break; }
      if (part == 0) tile_store<0>(p, st_tiles, m0, valid_nodes, va);
      else if (part == 1) tile_store<1>(p, st_tiles, m0, valid_nodes, va);
      else rows_store(st_tiles, rows_here, kcol, J, va);
      if (part < 2) tile_store<2>(p, st_tiles + kDwPieces * kDwTileBytes, j0, valid_nodes, vb);
      else rows_store(st_tiles + kDwPieces * kDwTileBytes, min(kDwTile, E - j0), kcol, J, vb);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy stores -> visible to the tensor core
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        tc_fence_after();
        const uint32_t a_addr = tiles_addr + stage * kDwStageBytes, b_addr = a_addr + kDwPieces * kDwTileBytes;
        // (piece of the input operand, piece of dz), the small products first: (0,2) (2,0) (1,1) (0,1) (1,0) (0,0)
#pragma unroll
        for (int k = 0; k < kDwBlock / 16; ++k)     // UMMA K = 16 bf16 = 32 bytes = 2 descriptor units
#pragma unroll
          for (int q = 0; q < 6; ++q) {
            const int pa = (0x010120 >> (4 * q)) & 0xF, pb = (0x001102 >> (4 * q)) & 0xF;
            umma_bf16(tmem_base, umma_desc(a_addr + pa * kDwTileBytes) + 2 * k,
                      umma_desc(b_addr + pb * kDwTileBytes) + 2 * k, idesc, !(b == 0 && k == 0 && q == 0));
          }
        umma_commit(stage_bar0 + 8 * stage);
        if (b == nblk - 1) umma_commit(acc_bar);
      }
    }
    if (failed) break;
    // the accumulator: tensor memory -> registers -> shared memory (whole rows) -> atomic adds of row segments
    const bool acc_ok = mbar_wait(acc_bar, items_done & 1u, &s_abort, p.wait_limit, p.st);
    if (__syncthreads_or(!acc_ok)) { failed = true; break; }
    ++items_done;
    tc_fence_after();
    constexpr int kRowStride = kDwTile + 4;                 // floats; 16-byte stores of a warp's 32 rows spread over all banks
    float* stage_out = reinterpret_cast<float*>(tiles);     // every MMA that read the operand stages has retired
    {
      const int quad = warp & 3, half = warp >> 2;          // a warp reads the tensor-memory lanes of quadrant (warp id mod 4)
      const int r = quad * 32 + lane;
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(half * 64);
      uint32_t v[64];
#pragma unroll
      for (int i = 0; i < 16; ++i) tmem_ld4(taddr + 4 * i, v + 4 * i);
      tmem_ld_wait();
      tc_fence_before();
      float* dst = stage_out + (size_t)r * kRowStride + half * 64;
#pragma unroll
      for (int i = 0; i < 16; ++i)
        *reinterpret_cast<float4*>(dst + 4 * i) = make_float4(__uint_as_float(v[4 * i]), __uint_as_float(v[4 * i + 1]),
                                                              __uint_as_float(v[4 * i + 2]), __uint_as_float(v[4 * i + 3]));
    }
    __syncthreads();
    const int rows_valid = part < 2 ? min(kDwTile, sh.rows[part] + 1 - m0) : rows_here;
    const int cols_valid = part < 2 ? min(kDwTile, J - j0) : min(kDwTile, E - j0);
    for (int r = warp; r < rows_valid; r += kDwThreads / 32) {
      float* out;
      if (part < 2) {
        const int f = m0 + r;
        out = f == sh.rows[part] ? p.db + j0 : p.dW + (size_t)((part ? E : 0) + f) * J + j0;
      } else {
        out = p.dEmb_rows + (size_t)s_ia[r] * E + j0;   // leaves with the same token share a row
      }
#pragma unroll
      for (int i = 0; i < kDwTile / 32; ++i) {
        const int c = lane + 32 * i;
        if (c < cols_valid) atomicAdd(out + c, stage_out[(size_t)r * kRowStride + c]);
      }
    }
    __syncthreads();   // the next item overwrites the index tables, the stages and the accumulator
  }
  // teardown: MMAs still in flight after a failed wait get a bounded time to retire before tensor memory goes back
  tc_fence_before();
  __syncthreads();
  if (failed && tid == 0) {
    umma_commit(drain_bar);
    mbar_drain(drain_bar, 0);
  }
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, kDwTile);
  }
}

}  // namespace

int init_dweight_tc_attributes(treelstm* ctx) {
  TL_CUDA(ctx, cudaFuncSetAttribute(k_bwd_dweight_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, kDwSmemBytes));
  return TREELSTM_OK;
}

// dW, db (and dEmb_rows, if given: then tok_slot holds every token's row) must have been cleared on the
// stream before; dz holds the gate gradients of every node.
int launch_dweight_tc(treelstm* ctx, int n, const int32_t* order, const int32_t* level_offset, const int32_t* token,
                      const int32_t* left, const int32_t* right, const float* h, const float* dz, float* dW, float* db,
                      const int* tok_slot, float* dEmb_rows, DevStatus* st, cudaStream_t stream) {
  DwParams p;
  p.n = n; p.n_leaves = 0; p.H = ctx->H; p.E = ctx->E; p.vocab = ctx->vocab; p.run = 0;
  p.order = order; p.level_offset = level_offset; p.token = token; p.left = left; p.right = right;
  p.emb = ctx->emb; p.h = h; p.dz = dz; p.W = ctx->W; p.dW = dW; p.db = db; p.st = st;
  p.tok_slot = tok_slot; p.dEmb_rows = dEmb_rows;
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  if (n == 0) return TREELSTM_OK;
  // The host does not know how the nodes divide into leaves and internal nodes (the level table stayed on the
  // device), so the kernel sizes its work items itself from the grid it finds: one CTA per SM unless even
  // single-block items are fewer (counted for the division that gives the most).
  int items = 0;
  for (int nl = 0; nl <= n; nl += (n > 8 ? n / 8 : 1)) {
    const DwShape s = dw_shape(n, nl, p.H, p.E, 1, dEmb_rows != nullptr);
    const int c = s.items[0] + s.items[1] + s.items[2];
    if (c > items) items = c;
  }
  const int grid = items < ctx->sm_count ? items : ctx->sm_count;
  k_bwd_dweight_tc<<<grid, kDwThreads, kDwSmemBytes, stream>>>(p);
  TL_CUDA(ctx, cudaGetLastError());
  ctx->launches += 1;
  return TREELSTM_OK;
}

}  // namespace tl
