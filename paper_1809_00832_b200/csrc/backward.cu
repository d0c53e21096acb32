// Training step: per-node softmax classifier + mean cross-entropy, then backpropagation through
// structure over the wavefronts in reverse (parents before children).
//
// Paper, Section 4.2.2: the gradient computation recurses at the same positions as the forward
// computation; Sections 4.2.1 / 5: a gradient operation needs the previous gradient and the
// forward values of its own node instance.  Here those values live in dense per-node arrays
// (gates, c, h) indexed by node id, so no lookup structure is needed and nothing can be routed
// to the wrong instance.
//
//   dh_n  = Wc (p_n - e_y)/N + [dIn from the caller]          dc_n = dc_caller*f + dh_n o (1 - tanh^2 c)
//   dz_o = dh tanh(c) o(1-o)   dz_i = dc u i(1-i)   dz_u = dc i (1-u^2)   dz_f* = dc c_* f*(1-f*)
//   dIn  = W dz  (rows [0,E): embedding row of a leaf; rows [E,E+2H): dh of the two children)
//   dW   = sum_n in_n (x) dz_n,   db = sum_n dz_n
#include "common.cuh"

namespace tl {

int ensure_host_levels(treelstm* ctx);  // api.cu

namespace {

constexpr unsigned kFull = 0xffffffffu;

struct BwdParams {
  int n, H, E, C, vocab, n_leaves;
  const int *left, *right, *token, *order, *labels;
  const float *emb, *W, *Wc, *bc, *h, *c, *gates;
  float *dh, *dc, *dz;
  float *loss, *dW, *db, *dWc, *dbc, *dEmb_rows;
  int *tok_slot, *touched_ids, *n_touched;
  int *pos_left, *pos_right;   // children of the node at every ready position (one-launch backward; scheduler scratch reused)
  DevStatus* st;
  long long* trace;   // cycle stamps of the one-launch backward (trace builds), else nullptr
};

// ---- touched embedding rows: flag, scan, compact ------------------------------------------- //
__global__ void k_bwd_mark_tokens(BwdParams p) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= p.n_leaves) return;
  p.tok_slot[chk(p.st, p.token[chk(p.st, p.order[r], p.n)], p.vocab)] = 1;  // level 0 occupies order[0 .. n_leaves)
}

// Exclusive scan of the flags over the vocabulary by one CTA; flagged ids are emitted in
// ascending order and tok_slot[id] becomes the row index of id in dEmb_rows.  A warp takes a
// contiguous run of 128-id groups: lane l holds ids 4 l .. 4 l + 3 of a group (one 16-byte load,
// eight groups in flight), four ballots per group (component c of every lane) kept in shared memory
// (s_mask, mask_cap words; groups beyond that are read again), a scan over the warps' counts, then
// a second pass that only stores.
// flags of ids id .. id + 3 (id a multiple of 4), zeros beyond the vocabulary or where `take` is false.  No
// branch: the compiler can then keep the loads of a batch in flight together.  The table has three
// spare entries behind its vocab + 1, so the last quad may be read whole.
__device__ __forceinline__ int4 load_flags4(const BwdParams& p, int id, bool take) {
  const int last_quad = ((p.vocab - 1) >> 2) << 2;
  int4 v = *reinterpret_cast<const int4*>(p.tok_slot + min(id, last_quad));
  v.x = take && id < p.vocab ? v.x : 0;
  v.y = take && id + 1 < p.vocab ? v.y : 0;
  v.z = take && id + 2 < p.vocab ? v.z : 0;
  v.w = take && id + 3 < p.vocab ? v.w : 0;
  return v;
}
__device__ void scan_tokens(const BwdParams& p, unsigned int* s_mask, int mask_cap) {   // blockDim a multiple of 32
  __shared__ int warp_sum[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  const int n_groups = (p.vocab + 127) / 128, per = (n_groups + nw - 1) / nw;
  const int g_lo = min(n_groups, warp * per), g_hi = min(n_groups, g_lo + per);
  constexpr int kBatch = 8;
  int count = 0;
  for (int g0 = g_lo; g0 < g_hi; g0 += kBatch) {
    int4 v[kBatch];
#pragma unroll
    for (int b = 0; b < kBatch; ++b)
      v[b] = load_flags4(p, (g0 + b) * 128 + 4 * lane, g0 + b < g_hi);
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const unsigned int m0 = __ballot_sync(kFull, v[b].x != 0), m1 = __ballot_sync(kFull, v[b].y != 0);
      const unsigned int m2 = __ballot_sync(kFull, v[b].z != 0), m3 = __ballot_sync(kFull, v[b].w != 0);
      if (g0 + b < g_hi) {
        if (4 * (g0 + b) + 3 < mask_cap && lane < 4) s_mask[4 * (g0 + b) + lane] = lane == 0 ? m0 : (lane == 1 ? m1 : (lane == 2 ? m2 : m3));
        count += __popc(m0) + __popc(m1) + __popc(m2) + __popc(m3);
      }
    }
  }
  if (lane == 0) warp_sum[warp] = count;
  TL_STAMP(tid == 0 ? p.trace : nullptr, kTraceLevels - 1, 9);    // first warp: flags read
  __syncthreads();
  TL_STAMP(tid == 0 ? p.trace : nullptr, kTraceLevels - 1, 10);   // all warps: flags read
  if (warp == 0) {
    int w = lane < nw ? warp_sum[lane] : 0, wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int t = __shfl_up_sync(kFull, wi, d);
      if (lane >= d) wi += t;
    }
    warp_sum[lane] = wi - w;
  }
  __syncthreads();
  int base = warp_sum[warp];
  const unsigned int below = (1u << lane) - 1u;
  for (int g = g_lo; g < g_hi; ++g) {
    const int id = g * 128 + 4 * lane;
    unsigned int m0, m1, m2, m3;
    if (4 * g + 3 < mask_cap) {
      const uint4 m = *reinterpret_cast<const uint4*>(s_mask + 4 * g);
      m0 = m.x; m1 = m.y; m2 = m.z; m3 = m.w;
    } else {
      const int4 v = load_flags4(p, id, true);
      m0 = __ballot_sync(kFull, v.x != 0); m1 = __ballot_sync(kFull, v.y != 0);
      m2 = __ballot_sync(kFull, v.z != 0); m3 = __ballot_sync(kFull, v.w != 0);
    }
    // ids ascend lane by lane, component by component
    const int f0 = (m0 >> lane) & 1u, f1 = (m1 >> lane) & 1u, f2 = (m2 >> lane) & 1u, f3 = (m3 >> lane) & 1u;
    const int e0 = base + __popc(m0 & below) + __popc(m1 & below) + __popc(m2 & below) + __popc(m3 & below);
    const int e1 = e0 + f0, e2 = e1 + f1, e3 = e2 + f2;
    if (id + 3 < p.vocab) {
      *reinterpret_cast<int4*>(p.tok_slot + id) = make_int4(e0, e1, e2, e3);
    } else {
      if (id < p.vocab) p.tok_slot[id] = e0;
      if (id + 1 < p.vocab) p.tok_slot[id + 1] = e1;
      if (id + 2 < p.vocab) p.tok_slot[id + 2] = e2;
    }
    if (f0) p.touched_ids[e0] = id;       // a set flag implies id < vocab: flags beyond it were read as 0
    if (f1) p.touched_ids[e1] = id + 1;
    if (f2) p.touched_ids[e2] = id + 2;
    if (f3) p.touched_ids[e3] = id + 3;
    base += __popc(m0) + __popc(m1) + __popc(m2) + __popc(m3);
  }
  if (warp == nw - 1 && lane == 0) { *p.n_touched = base; p.st->n_touched = base; }
}
// The same scan spread over the CTAs of the one-launch backward, in two steps with a grid barrier between
// them: scan_count_groups writes the number of flagged ids of every 128-id group to group_count[], then
// scan_place_groups sums the counts before a group and places its ids.  Group g belongs to warp 0 of CTA
// gridDim.x - 1 - g % gridDim.x: the high-numbered CTAs, which have no block in a narrow wavefront, so that
// the second step runs beside the first wavefronts instead of ahead of them.
__device__ __forceinline__ void scan_count_groups(const BwdParams& p, int* group_count) {
  if (threadIdx.x >= 32) return;
  const int lane = threadIdx.x, n_groups = (p.vocab + 127) / 128;
  for (int g = (int)(gridDim.x - 1 - blockIdx.x); g < n_groups; g += (int)gridDim.x) {
    const int4 v = load_flags4(p, g * 128 + 4 * lane, true);
    const int c = __popc(__ballot_sync(kFull, v.x != 0)) + __popc(__ballot_sync(kFull, v.y != 0)) +
                  __popc(__ballot_sync(kFull, v.z != 0)) + __popc(__ballot_sync(kFull, v.w != 0));
    if (lane == 0) group_count[g] = c;
  }
}
__device__ __forceinline__ void scan_place_groups(const BwdParams& p, const int* group_count) {
  if (threadIdx.x >= 32) return;
  const int lane = threadIdx.x, n_groups = (p.vocab + 127) / 128;
  const unsigned int below = (1u << lane) - 1u;
  for (int g = (int)(gridDim.x - 1 - blockIdx.x); g < n_groups; g += (int)gridDim.x) {
    const int id = g * 128 + 4 * lane;
    const int4 v = load_flags4(p, id, true);          // the group's flags: nobody else touches them
    int base = 0;
    for (int q = lane; q < g; q += 32) base += group_count[q];
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) base += __shfl_xor_sync(kFull, base, d);
    const unsigned int m0 = __ballot_sync(kFull, v.x != 0), m1 = __ballot_sync(kFull, v.y != 0);
    const unsigned int m2 = __ballot_sync(kFull, v.z != 0), m3 = __ballot_sync(kFull, v.w != 0);
    const int f0 = (m0 >> lane) & 1u, f1 = (m1 >> lane) & 1u, f2 = (m2 >> lane) & 1u, f3 = (m3 >> lane) & 1u;
    const int e0 = base + __popc(m0 & below) + __popc(m1 & below) + __popc(m2 & below) + __popc(m3 & below);
    const int e1 = e0 + f0, e2 = e1 + f1, e3 = e2 + f2;
    if (id + 3 < p.vocab) {
      *reinterpret_cast<int4*>(p.tok_slot + id) = make_int4(e0, e1, e2, e3);
    } else {
      if (id < p.vocab) p.tok_slot[id] = e0;
      if (id + 1 < p.vocab) p.tok_slot[id + 1] = e1;
      if (id + 2 < p.vocab) p.tok_slot[id + 2] = e2;
    }
    if (f0) p.touched_ids[e0] = id;
    if (f1) p.touched_ids[e1] = id + 1;
    if (f2) p.touched_ids[e2] = id + 2;
    if (f3) p.touched_ids[e3] = id + 3;
    if (g == n_groups - 1 && lane == 0) {
      const int total = base + __popc(m0) + __popc(m1) + __popc(m2) + __popc(m3);
      *p.n_touched = total; p.st->n_touched = total;
    }
  }
}
constexpr int kScanMaskWords = 8192;
__global__ void __launch_bounds__(1024) k_bwd_scan_tokens(BwdParams p) {
  __shared__ __align__(16) unsigned int s_mask[kScanMaskWords];
  scan_tokens(p, s_mask, kScanMaskWords);
}

// ---- classifier: logits, softmax, loss, dlogits, dh (classifier part), dWc, dbc -------------- //
// One warp per node: the lanes share the contraction over h (lane j takes units j, j + 32, ...),
// a butterfly sum gives every lane all logits, lane k keeps class k (C <= 32).
constexpr int kClsWarps = 8;
constexpr int kClsNodesPerCta = 8;    // one node per warp and group: the chains of dependent loads of a node are long

// The CTA takes the node groups vb_first, vb_first + vb_step, ...; s_dWc [H][C] + [C] collects its partial sums.
__device__ void classifier_groups(const BwdParams& p, int vb_first, int vb_step, float* s_dWc) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = p.H, C = p.C;
  for (int i = tid; i < H * C + C; i += blockDim.x) s_dWc[i] = 0.f;
  __syncthreads();
#ifdef TREELSTM_TRACE
  long long* const ctrace = blockIdx.x == 1 && tid == 0 ? p.trace : nullptr;   // the first CTA with nodes to classify
#endif
  TL_STAMP(ctrace, kTraceLevels - 1, 11);
  const float inv_n = 1.0f / (float)p.n;
  const int n_groups = (p.n + kClsNodesPerCta - 1) / kClsNodesPerCta;
  for (int vb = vb_first; vb < n_groups; vb += vb_step)
  for (int q = warp; q < kClsNodesPerCta; q += kClsWarps) {
    const int node0 = vb * kClsNodesPerCta;
    const int node = node0 + q;
    if (node >= p.n) break;
    const float* hn = p.h + (size_t)node * H;
    const int y = p.labels[node];                       // asked for now: they arrive with the first h values
    const float my_bias = lane < C ? __ldg(p.bc + lane) : 0.f;
    float logit = -INFINITY;
    for (int k = 0; k < C; ++k) {
      float part = 0.f;
      for (int j = lane; j < H; j += 32) part = fmaf(hn[j], __ldg(p.Wc + j * C + k), part);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(kFull, part, d);
      if (lane == k) logit = part + my_bias;
    }
    float m = logit;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, d));
    float e = lane < C ? expf(logit - m) : 0.f, sum = e;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(kFull, sum, d);
    const bool y_ok = y >= 0 && y < C;
    if (!y_ok && lane == 0) report(p.st, TREELSTM_ERR_LABEL_OUT_OF_RANGE);
    const float lse = m + logf(sum);
    const float logit_y = __shfl_sync(kFull, logit, y_ok ? y : 0);
    if (lane == 0 && y_ok) atomicAdd(p.loss, (lse - logit_y) * inv_n);
    const float dlogit = lane < C ? (e / sum - (lane == y ? 1.f : 0.f)) * inv_n : 0.f;
    if (lane < C) atomicAdd(&s_dWc[H * C + lane], dlogit);
    for (int j0 = 0; j0 < H; j0 += 32) {
      const int j = j0 + lane;
      const float hj = j < H ? hn[j] : 0.f;
      float dhj = 0.f;
      for (int k = 0; k < C; ++k) {
        const float dk = __shfl_sync(kFull, dlogit, k);
        if (j < H) {
          dhj = fmaf(p.Wc[j * C + k], dk, dhj);
          atomicAdd(&s_dWc[j * C + k], hj * dk);
        }
      }
      if (j < H) p.dh[(size_t)node * H + j] = dhj;
    }
    TL_STAMP(ctrace, kTraceLevels - 1, 12);   // first warp: a node done
  }
  __syncthreads();
  TL_STAMP(ctrace, kTraceLevels - 1, 13);     // all warps: nodes done
  if (vb_first >= n_groups) return;   // a CTA without a group has nothing to add (and 300 CTAs adding zeros to the same H x C words queue up)
  for (int i = tid; i < H * C; i += blockDim.x) atomicAdd(&p.dWc[i], s_dWc[i]);
  for (int i = tid; i < C; i += blockDim.x) atomicAdd(&p.dbc[i], s_dWc[H * C + i]);
  TL_STAMP(ctrace, kTraceLevels - 1, 14);     // partial sums sent
}
__global__ void __launch_bounds__(kClsWarps * 32) k_bwd_classifier(BwdParams p) {
  extern __shared__ float s_dyn[];
  classifier_groups(p, blockIdx.x, gridDim.x, s_dyn);
}

// ---- gate gradients of one wavefront -------------------------------------------------------- //
__device__ __forceinline__ void gates_element(const BwdParams& p, int row_begin, long long idx, int leaf) {
  const int H = p.H;
  const int row = row_begin + (int)(idx / H), u = (int)(idx % H);
  const int node = chk(p.st, p.order[row], p.n);
  const float* g = p.gates + (size_t)node * 5 * H + u;
  const float gi = g[0], go = g[3 * H], gu = g[4 * H];
  const float cn = p.c[(size_t)node * H + u];
  const float tc = tanhf(cn);
  const float dhn = p.dh[(size_t)node * H + u];
  const float dcn = p.dc[(size_t)node * H + u] + dhn * go * (1.f - tc * tc);
  float* dz = p.dz + (size_t)node * 5 * H + u;
  dz[0] = dcn * gu * gi * (1.f - gi);
  dz[3 * H] = dhn * tc * go * (1.f - go);
  dz[4 * H] = dcn * gi * (1.f - gu * gu);
  if (leaf) {
    dz[H] = 0.f;
    dz[2 * H] = 0.f;
  } else {
    const int l = chk(p.st, p.left[node], p.n), r = chk(p.st, p.right[node], p.n);
    const float gfl = g[H], gfr = g[2 * H];
    dz[H] = dcn * p.c[(size_t)l * H + u] * gfl * (1.f - gfl);
    dz[2 * H] = dcn * p.c[(size_t)r * H + u] * gfr * (1.f - gfr);
    p.dc[(size_t)l * H + u] = dcn * gfl;  // every node has exactly one caller: plain stores
    p.dc[(size_t)r * H + u] = dcn * gfr;
  }
}
__global__ void k_bwd_gates(BwdParams p, int row_begin, int row_end, int leaf) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx < (long long)(row_end - row_begin) * p.H) gates_element(p, row_begin, idx, leaf);
}

// ---- dIn = dz W^T for one wavefront --------------------------------------------------------- //
// out[row][k] = sum_j dz[row][j] * W[koff + k][j]; tile 64 rows x 64 outputs, 16 x 16 threads.
// The next chunk of the contraction is fetched into registers while the current one is
// multiplied out of shared memory (two buffers, one CTA barrier per chunk).
constexpr int BT = 64, BK = 32;
constexpr int kLd = BT * BK / 256;   // elements of each operand per thread and chunk

constexpr int kDiRow = BK + 4;       // row stride: float4 reads along the contraction, 16 rows spread over all banks
struct DinputSmem {
  __align__(16) float As[2][BT][kDiRow];
  __align__(16) float Bs[2][BT][kDiRow];
  int node[BT];
  int dst_a[BT], dst_b[BT];   // where a row's dIn goes: left / right child, or (leaves) its row of dEmb_rows
  int fnode[2][BT], fleft[2][BT], fright[2][BT];   // the same for the blocks of dinput_fused: two sets used in turn
};
__device__ void dinput_block(const BwdParams& p, int row_begin, int row_end, int leaf, int bx, int by, int nby,
                             DinputSmem& sm) {
  float (*As)[BT][kDiRow] = sm.As;
  float (*Bs)[BT][kDiRow] = sm.Bs;
  int* s_node = sm.node;
  const int H = p.H, E = p.E, J = 5 * H;
  const int K = leaf ? E : 2 * H, koff = leaf ? 0 : E;
  const int tiles_k = (K + BT - 1) / BT;
  const int row0 = row_begin + (bx / tiles_k) * BT, k0 = (bx % tiles_k) * BT;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  __syncthreads();   // a previous block of this CTA may still be reading the shared arrays
  // the index chains (order -> children, or order -> token -> touched row) are resolved once per block
  for (int i = tid; i < BT; i += 256) {
    int node = -1, da = 0, db = 0;
    if (row0 + i < row_end) {
      node = chk(p.st, p.order[row0 + i], p.n);
      if (leaf) da = chk(p.st, p.tok_slot[chk(p.st, p.token[node], p.vocab)], p.n_leaves);
      else { da = chk(p.st, p.left[node], p.n); db = chk(p.st, p.right[node], p.n); }
    }
    s_node[i] = node; sm.dst_a[i] = da; sm.dst_b[i] = db;
  }
  __syncthreads();
  float acc[4][4] = {};
  float ra[kLd], rb[kLd];
  // Loads without a branch (rows and columns outside the block clamped onto valid ones); what they brought for
  // elements outside is replaced by zeros at the store - a use right behind the loads would make the
  // multiply-adds of the current chunk wait for them.
  auto fetch = [&](int j0) {
#pragma unroll
    for (int q = 0; q < kLd; ++q) {
      const int e = tid + q * 256, i = e / BK, j = min(j0 + e % BK, J - 1);
      ra[q] = p.dz[(size_t)max(s_node[i], 0) * J + j];
      rb[q] = __ldg(p.W + (size_t)(koff + min(k0 + i, K - 1)) * J + j);
    }
  };
  auto stash = [&](int buf, int j0) {
#pragma unroll
    for (int q = 0; q < kLd; ++q) {
      const int e = tid + q * 256, i = e / BK, j = j0 + e % BK;
      As[buf][i][e % BK] = (s_node[i] >= 0 && j < J) ? ra[q] : 0.f;
      Bs[buf][i][e % BK] = (k0 + i < K && j < J) ? rb[q] : 0.f;
    }
  };
  // gridDim.y CTAs share the contraction: each takes a contiguous run of chunks and adds its
  // partial sums with atomics (few levels fill the GPU on their own, the chain of dependent
  // memory round trips per CTA is what costs time)
  const int chunks_all = (J + BK - 1) / BK;
  const int per_split = (chunks_all + nby - 1) / nby;
  const int c_lo = by * per_split, chunks = min(chunks_all, c_lo + per_split);
  if (c_lo >= chunks) return;
  fetch(c_lo * BK);
  stash(c_lo & 1, c_lo * BK);
  __syncthreads();
  for (int cidx = c_lo; cidx < chunks; ++cidx) {
    const int buf = cidx & 1;
    if (cidx + 1 < chunks) fetch((cidx + 1) * BK);
#pragma unroll
    for (int jj = 0; jj < BK; jj += 4) {
      float4 a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        a[i] = *reinterpret_cast<const float4*>(&As[buf][ty + 16 * i][jj]);
        b[i] = *reinterpret_cast<const float4*>(&Bs[buf][tx + 16 * i][jj]);
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          acc[i][q] = fmaf(a[i].x, b[q].x, acc[i][q]);
          acc[i][q] = fmaf(a[i].y, b[q].y, acc[i][q]);
          acc[i][q] = fmaf(a[i].z, b[q].z, acc[i][q]);
          acc[i][q] = fmaf(a[i].w, b[q].w, acc[i][q]);
        }
    }
    if (cidx + 1 < chunks) stash(buf ^ 1, (cidx + 1) * BK);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int node = s_node[ty + 16 * i];
    if (node < 0) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int k = k0 + tx + 16 * q;
      if (k >= K) continue;
      if (leaf) {
        atomicAdd(&p.dEmb_rows[(size_t)sm.dst_a[ty + 16 * i] * E + k], acc[i][q]);
      } else {
        const int child = k < H ? sm.dst_a[ty + 16 * i] : sm.dst_b[ty + 16 * i];
        atomicAdd(&p.dh[(size_t)child * H + (k < H ? k : k - H)], acc[i][q]);
      }
    }
  }
}
// How many CTAs share the contraction of one dIn tile.  A 64 x 64 tile costs about 4 k cycles per
// 32-wide chunk of the contraction whatever the number of valid rows, so a wavefront with few tiles
// spreads the chunks over as many CTAs as there are (about two per SM), down to one chunk each.
__host__ __device__ inline int dinput_splits(int tiles, int J) {
  const int chunks_all = (J + BK - 1) / BK;
  if (tiles >= 148) return 1;
  int s = 296 / (tiles > 0 ? tiles : 1);
  if (s < 6) s = 6;
  return s < chunks_all ? s : chunks_all;
}
__host__ __device__ inline int dinput_tiles(int rows, int K) { return ((rows + BT - 1) / BT) * ((K + BT - 1) / BT); }
__global__ void __launch_bounds__(256)
k_bwd_dinput(BwdParams p, int row_begin, int row_end, int leaf) {
  __shared__ DinputSmem sm;
  dinput_block(p, row_begin, row_end, leaf, blockIdx.x, blockIdx.y, gridDim.y, sm);
}

// ---- narrow internal wavefronts of the one-launch backward: gate gradients inside the contraction -- //
// A block of dIn = dz W^T forms the dz values of its chunk itself instead of reading them back, so a
// narrow wavefront needs neither a pass of its own for the gate gradients nor the grid barrier behind
// it.  What does not depend on the wavefront above - the rows' index triples (node, left, right; kept
// by position in pos_left / pos_right, filled once at the start) and the weight chunk - is asked for
// with cp.async before the CTA enters the grid barrier and lands in shared memory while it waits;
// after the barrier one round of loads brings dh, dc (just written by the wavefront above) together
// with the forward's gate activations and cell states.  Same expressions as gates_element.  The
// blocks of the first output tile (k0 == 0) also store dz for the dW contraction and hand dc to the
// children; every (node, gate column) belongs to exactly one of them.
struct FusedItem {
  int row0, rows, k0, c_lo, chunks;   // first row (position in the ready order), valid rows, first output, chunk range
};
__device__ __forceinline__ FusedItem fused_item(const BwdParams& p, int row_begin, int row_end, int bx, int by, int nby) {
  const int K = 2 * p.H, J = 5 * p.H;
  const int tiles_k = (K + BT - 1) / BT;
  const int chunks_all = (J + BK - 1) / BK, per_split = (chunks_all + nby - 1) / nby;
  FusedItem it;
  it.row0 = row_begin + (bx / tiles_k) * BT;
  it.rows = min(BT, row_end - it.row0);
  it.k0 = (bx % tiles_k) * BT;
  it.c_lo = by * per_split;
  it.chunks = min(chunks_all, it.c_lo + per_split);
  return it;
}
// What a block needs that does not depend on the wavefront above, fetched into registers (a 4-byte cp.async
// per element measured ~130 cycles of issue each: slower than holding nine registers across the barrier) ...
struct FusedFetch {
  int idx;          // thread t < 192: order / pos_left / pos_right of row t % 64
  float w[kLd];     // the thread's elements of the first weight chunk
};
__device__ __forceinline__ void fused_fetch(const BwdParams& p, const FusedItem& it, int j0, FusedFetch& f) {
  const int J = 5 * p.H, K = 2 * p.H, t = threadIdx.x;
  f.idx = 0;
  if (t < 3 * BT) {
    const int which = t / BT, i = t % BT;
    const int pos = it.row0 + min(i, it.rows - 1);
    f.idx = *(which == 0 ? p.order + pos : (which == 1 ? p.pos_left + pos : p.pos_right + pos));
  }
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = t + q * 256, i = min(it.k0 + e / BK, K - 1), j = min(j0 + e % BK, J - 1);
    f.w[q] = __ldg(p.W + (size_t)(p.E + i) * J + j);
  }
}
// ... and put into index set `ib` and operand buffer `buf` (a CTA barrier must follow)
__device__ __forceinline__ void fused_deposit(const BwdParams& p, const FusedItem& it, DinputSmem& sm, int ib, int buf,
                                              int j0, const FusedFetch& f) {
  const int J = 5 * p.H, K = 2 * p.H, t = threadIdx.x;
  if (t < 3 * BT) {
    const int which = t / BT, i = t % BT;
    *(which == 0 ? &sm.fnode[ib][i] : (which == 1 ? &sm.fleft[ib][i] : &sm.fright[ib][i])) = f.idx;
  }
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = t + q * 256;
    sm.Bs[buf][e / BK][e % BK] = (it.k0 + e / BK < K && j0 + e % BK < J) ? f.w[q] : 0.f;
  }
}
// weight chunk j0 of the block into operand buffer `buf` (later chunks of a block)
__device__ __forceinline__ void fused_weights(const BwdParams& p, const FusedItem& it, DinputSmem& sm, int buf, int j0) {
  const int J = 5 * p.H, K = 2 * p.H, t = threadIdx.x;
  float w[kLd];
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = t + q * 256, i = min(it.k0 + e / BK, K - 1), j = min(j0 + e % BK, J - 1);
    w[q] = __ldg(p.W + (size_t)(p.E + i) * J + j);
  }
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = t + q * 256;
    sm.Bs[buf][e / BK][e % BK] = (it.k0 + e / BK < K && j0 + e % BK < J) ? w[q] : 0.f;
  }
}
__device__ __forceinline__ int gate_of_column(int j, int H) { return (j >= H) + (j >= 2 * H) + (j >= 3 * H) + (j >= 4 * H); }
// dz values of chunk j0 for the block's rows -> operand buffer `buf`.  All loads first and without a
// branch (rows and columns beyond the block are clamped onto valid ones and discarded afterwards), so that
// they are in flight together: one round trip instead of one per element; then the arithmetic and the stores.
__device__ __forceinline__ void fused_gate_gradients(const BwdParams& p, const FusedItem& it, DinputSmem& sm, int ib,
                                                     int buf, int j0) {
  const int H = p.H, J = 5 * H, tid = threadIdx.x;
  float dhn[kLd], dci[kLd], go[kLd], cn[kLd], g1[kLd], g2[kLd];
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = tid + q * 256, i = min(e / BK, it.rows - 1), j = min(j0 + e % BK, J - 1);
    const int node = chk(p.st, sm.fnode[ib][i], p.n);
    const int g = gate_of_column(j, H), u = j - g * H;
    const bool forget = g == 1 || g == 2;
    const int child = chk(p.st, g == 2 ? sm.fright[ib][i] : sm.fleft[ib][i], p.n);
    const float* gt = p.gates + (size_t)node * J + u;
    dhn[q] = p.dh[(size_t)node * H + u];
    dci[q] = p.dc[(size_t)node * H + u];
    go[q] = gt[3 * H];
    cn[q] = p.c[(size_t)node * H + u];
    g1[q] = gt[forget ? g * H : 0];                                   // f_l / f_r, else i
    g2[q] = *(forget ? p.c + (size_t)child * H + u : gt + 4 * H);    // the child's cell state, else u
  }
  const bool keep = it.k0 == 0;
#pragma unroll
  for (int q = 0; q < kLd; ++q) {
    const int e = tid + q * 256, i = e / BK, j = j0 + e % BK;
    float dz = 0.f;
    if (i < it.rows && j < J) {
      const int node = chk(p.st, sm.fnode[ib][i], p.n);
      const int g = gate_of_column(j, H), u = j - g * H;
      const float tc = tanhf(cn[q]);
      const float dcn = dci[q] + dhn[q] * go[q] * (1.f - tc * tc);
      if (g == 3) {
        dz = dhn[q] * tc * go[q] * (1.f - go[q]);
      } else if (g == 1 || g == 2) {
        const float gf = g1[q];
        dz = dcn * g2[q] * gf * (1.f - gf);
        if (keep) p.dc[(size_t)chk(p.st, g == 1 ? sm.fleft[ib][i] : sm.fright[ib][i], p.n) * H + u] = dcn * gf;
      } else {
        const float gi = g1[q], gu = g2[q];
        dz = g == 0 ? dcn * gu * gi * (1.f - gi) : dcn * gi * (1.f - gu * gu);
      }
      if (keep) p.dz[(size_t)node * J + j] = dz;
    }
    sm.As[buf][i][e % BK] = dz;
  }
}
// one chunk of the contraction for the first 16 NI rows of the tile (thread (tx, ty): rows ty + 16 i, outputs tx + 16 q)
template <int NI>
__device__ __forceinline__ void fused_chunk(const DinputSmem& sm, int buf, int tx, int ty, float (&acc)[4][4]) {
#pragma unroll
  for (int jj = 0; jj < BK; jj += 4) {
    float4 a[NI], b[4];
#pragma unroll
    for (int i = 0; i < NI; ++i) a[i] = *reinterpret_cast<const float4*>(&sm.As[buf][ty + 16 * i][jj]);
#pragma unroll
    for (int q = 0; q < 4; ++q) b[q] = *reinterpret_cast<const float4*>(&sm.Bs[buf][tx + 16 * q][jj]);
#pragma unroll
    for (int i = 0; i < NI; ++i)
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        acc[i][q] = fmaf(a[i].x, b[q].x, acc[i][q]);
        acc[i][q] = fmaf(a[i].y, b[q].y, acc[i][q]);
        acc[i][q] = fmaf(a[i].z, b[q].z, acc[i][q]);
        acc[i][q] = fmaf(a[i].w, b[q].w, acc[i][q]);
      }
  }
}
// One block.  fetched: `f` holds the block's index triples and first weight chunk (fused_fetch was called before
// the grid barrier) and no thread of the CTA still reads the operand buffers.
// buffers_free() runs once, when the block no longer needs the operand buffers and before its results go out.
template <class FreeFn>
__device__ __forceinline__ void dinput_fused(const BwdParams& p, const FusedItem& it, DinputSmem& sm, int ib, bool fetched,
                                             FusedFetch& f, long long* trace, int lvl, FreeFn buffers_free) {
  (void)trace; (void)lvl;
  if (it.c_lo >= it.chunks) { buffers_free(); return; }   // the same for every thread of the CTA
  const int H = p.H, K = 2 * H;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  if (!fetched) {
    __syncthreads();   // a previous block of this CTA may still be reading the shared arrays
    fused_fetch(p, it, it.c_lo * BK, f);
  }
  fused_deposit(p, it, sm, ib, it.c_lo & 1, it.c_lo * BK, f);
  __syncthreads();
  TL_STAMP(trace, lvl, 8);   // index triples and first weight chunk in shared memory
  float acc[4][4] = {};
  fused_gate_gradients(p, it, sm, ib, it.c_lo & 1, it.c_lo * BK);
  __syncthreads();
  TL_STAMP(trace, lvl, 5);   // gate gradients of the first chunk formed by all warps
  const int ni = (it.rows + 15) / 16;   // 16-row groups of the tile that hold nodes
  for (int cidx = it.c_lo; cidx < it.chunks; ++cidx) {
    const int buf = cidx & 1;
    const bool more = cidx + 1 < it.chunks;
    if (more) fused_weights(p, it, sm, buf ^ 1, (cidx + 1) * BK);
    if (ni == 1) fused_chunk<1>(sm, buf, tx, ty, acc);
    else if (ni == 2) fused_chunk<2>(sm, buf, tx, ty, acc);
    else if (ni == 3) fused_chunk<3>(sm, buf, tx, ty, acc);
    else fused_chunk<4>(sm, buf, tx, ty, acc);
    if (more) {
      fused_gate_gradients(p, it, sm, ib, buf ^ 1, (cidx + 1) * BK);
    }
    __syncthreads();
  }
  TL_STAMP(trace, lvl, 6);   // contraction done
  buffers_free();
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty + 16 * i;
    if (r >= it.rows) continue;
    const int l = chk(p.st, sm.fleft[ib][r], p.n), rr = chk(p.st, sm.fright[ib][r], p.n);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int k = it.k0 + tx + 16 * q;
      if (k >= K) continue;
      atomicAdd(&p.dh[(size_t)(k < H ? l : rr) * H + (k < H ? k : k - H)], acc[i][q]);
    }
  }
}

// ---- dW = In^T dZ (contraction over nodes) and db ------------------------------------------- //
// part 0: rows [0,E) from the leaves (In = embedding rows); part 1: rows [E,E+2H) from the
// internal nodes (In = [h_l | h_r]).  Tile 64 (k) x 64 (j); gridDim.y splits the node range.
constexpr int WR = 32;               // nodes per chunk: enough multiply-adds per chunk to cover the fetch of the next one
constexpr int kLdW = WR * BT / 256;  // elements of each operand per thread and chunk

constexpr int kDwRows = 128;         // nodes per block of the dW contraction
struct DweightSmem {
  __align__(16) float As[2][WR][BT];
  __align__(16) float Bs[2][WR][BT];
  int node[kDwRows], ia[kDwRows], ib[kDwRows];   // node id and where its operand row comes from
};
__device__ void dweight_block(const BwdParams& p, int part, int row_begin, int row_end, int rows_per_split,
                              int bx, int by, DweightSmem& sm) {
  float (*As)[WR][BT] = sm.As;
  float (*Bs)[WR][BT] = sm.Bs;
  const int H = p.H, E = p.E, J = 5 * H;
  const int K = part == 0 ? E : 2 * H, koff = part == 0 ? 0 : E;
  const int tiles_j = (J + BT - 1) / BT;
  const int k0 = (bx / tiles_j) * BT, j0 = (bx % tiles_j) * BT;
  const int r_lo = row_begin + by * rows_per_split;
  __syncthreads();   // a previous block of this CTA may still be reading the shared arrays
  const int r_hi = min(row_end, r_lo + min(rows_per_split, kDwRows));
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // the index chain order -> token / children is resolved once per block, not once per fetched element
  for (int i = tid; i < kDwRows; i += 256) {
    int node = 0, ia = 0, ib = 0;
    if (r_lo + i < r_hi) {
      node = chk(p.st, p.order[r_lo + i], p.n);
      if (part == 0) ia = chk(p.st, p.token[node], p.vocab);
      else { ia = chk(p.st, p.left[node], p.n); ib = chk(p.st, p.right[node], p.n); }
    }
    sm.node[i] = node; sm.ia[i] = ia; sm.ib[i] = ib;
  }
  __syncthreads();
  float acc[4][4] = {};
  float ra[kLdW], rb[kLdW];
  // element e of a chunk: node rr = e / 64 of the chunk, column cc = e % 64 of the tile
  auto fetch = [&](int r0) {
#pragma unroll
    for (int q = 0; q < kLdW; ++q) {
      const int e = tid + q * 256, rr = e / BT, cc = e % BT;
      const int row = r0 + rr;
      float va = 0.f, vb = 0.f;
      if (row < r_hi) {
        const int li = row - r_lo;
        const int k = k0 + cc, j = j0 + cc;
        if (k < K) {
          if (part == 0) va = __ldg(p.emb + (size_t)sm.ia[li] * E + k);
          else va = k < H ? p.h[(size_t)sm.ia[li] * H + k] : p.h[(size_t)sm.ib[li] * H + (k - H)];
        }
        if (j < J) vb = p.dz[(size_t)sm.node[li] * J + j];
      }
      ra[q] = va;
      rb[q] = vb;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int q = 0; q < kLdW; ++q) {
      const int e = tid + q * 256;
      As[buf][e / BT][e % BT] = ra[q];
      Bs[buf][e / BT][e % BT] = rb[q];
    }
  };
  if (r_lo < r_hi) {
    fetch(r_lo);
    stash(0);
  }
  __syncthreads();
  int buf = 0;
  for (int r0 = r_lo; r0 < r_hi; r0 += WR, buf ^= 1) {
    if (r0 + WR < r_hi) fetch(r0 + WR);
#pragma unroll
    for (int rr = 0; rr < WR; ++rr) {   // thread (tx, ty): outputs k0 + 4 ty .. + 3  x  j0 + 4 tx .. + 3
      const float4 a4 = *reinterpret_cast<const float4*>(&As[buf][rr][4 * ty]);
      const float4 b4 = *reinterpret_cast<const float4*>(&Bs[buf][rr][4 * tx]);
      const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int q = 0; q < 4; ++q) acc[i][q] = fmaf(a[i], b[q], acc[i][q]);
    }
    if (r0 + WR < r_hi) stash(buf ^ 1);
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int k = k0 + 4 * ty + i;
    if (k >= K) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int j = j0 + 4 * tx + q;
      if (j < J) atomicAdd(&p.dW[(size_t)(koff + k) * J + j], acc[i][q]);
    }
  }
}
__global__ void __launch_bounds__(256)
k_bwd_dweight(BwdParams p, int part, int row_begin, int row_end, int rows_per_split) {
  __shared__ DweightSmem sm;
  dweight_block(p, part, row_begin, row_end, rows_per_split, blockIdx.x, blockIdx.y, sm);
}

// column j of db over the nodes [256 by, 256 by + 256)
__device__ __forceinline__ void dbias_piece(const BwdParams& p, int j, int by) {
  const int J = 5 * p.H;
  const int r_lo = by * 256, r_hi = min(p.n, r_lo + 256);
  float acc = 0.f;
  for (int r = r_lo; r < r_hi; ++r) acc += p.dz[(size_t)r * J + j];
  atomicAdd(&p.db[j], acc);
}
__global__ void k_bwd_dbias(BwdParams p) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < 5 * p.H) dbias_piece(p, j, blockIdx.y);
}

// ---- the whole backward pass in one cooperative launch --------------------------------------- //
// Used after a forward that left the level table on the device only (persistent / sub-forest
// modes): no host round trip, no launch per wavefront.  Phases, separated by the bounded grid
// barrier: clear the outputs | mark leaf tokens | token scan (CTA 0) next to the classifier (all
// other CTAs) | per wavefront from the top: gate gradients, then dIn = dz W^T into the children |
// dW, db (they only need every dz).
constexpr int kFusedMaxRows = 128;   // widest wavefront whose gate gradients are formed inside the contraction
#ifdef TREELSTM_TRACE
#define TL_TRACE_ARG trace
#else
#define TL_TRACE_ARG nullptr
#endif
union BwdSmem {
  DinputSmem di;
  DweightSmem dw;
};
template <class T>
__device__ __forceinline__ void zero_range(T* ptr, size_t count, size_t gtid, size_t gthreads) {
  for (size_t i = gtid; i < count; i += gthreads) ptr[i] = T(0);
}
__global__ void __launch_bounds__(256, 2)
k_bwd_persistent(BwdParams p, const int* level_offset, long long wait_limit, int with_dweight) {
  extern __shared__ float4 s_dyn4[];
  BwdSmem& sm = *reinterpret_cast<BwdSmem*>(s_dyn4);
  float* s_cls = reinterpret_cast<float*>(s_dyn4) + (sizeof(BwdSmem) + 3) / 4;
  __shared__ int s_flag;
  if (ld_volatile(&p.st->status) != 0) return;
  const int n_levels = p.st->n_levels;
  const int n = p.n, H = p.H, E = p.E, C = p.C, J = 5 * H;
#ifdef TREELSTM_TRACE
  // first CTA, first thread: row l of the stamp table = wavefront l (slot 0 start, 1 gate gradients done,
  // 2 barrier, 3 input gradients done, 4 barrier); last row = phases of the kernel
  long long* const trace = blockIdx.x == 0 && threadIdx.x == 0 ? p.trace : nullptr;
#endif
  TL_STAMP(trace, kTraceLevels - 1, 0);
  p.n_leaves = n_levels > 0 ? level_offset[1] : 0;
  const size_t gtid = (size_t)blockIdx.x * blockDim.x + threadIdx.x, gthreads = (size_t)gridDim.x * blockDim.x;
  unsigned int arrivals = 0;
  auto barrier = [&]() {
    arrivals += gridDim.x;
    return grid_barrier(p.st, arrivals, wait_limit, &s_flag, true, &p.st->barrier_bwd);
  };
  if (gtid == 0) { *p.loss = 0.f; *p.n_touched = 0; }
  zero_range(p.dW, (size_t)(E + 2 * H) * J, gtid, gthreads);
  zero_range(p.db, (size_t)J, gtid, gthreads);
  zero_range(p.dWc, (size_t)H * C, gtid, gthreads);
  zero_range(p.dbc, (size_t)C, gtid, gthreads);
  zero_range(p.dc, (size_t)n * H, gtid, gthreads);
  zero_range(p.tok_slot, (size_t)p.vocab + 1, gtid, gthreads);
  zero_range(p.dEmb_rows, (size_t)p.n_leaves * E, gtid, gthreads);
  if (!barrier()) return;
  TL_STAMP(trace, kTraceLevels - 1, 1);   // outputs and scratch cleared
  for (size_t r = gtid; r < (size_t)p.n_leaves; r += gthreads)
    p.tok_slot[chk(p.st, p.token[chk(p.st, p.order[r], p.n)], p.vocab)] = 1;
  for (size_t r = (size_t)p.n_leaves + gtid; r < (size_t)n; r += gthreads) {   // children by ready position
    const int node = chk(p.st, p.order[r], p.n);
    p.pos_left[r] = p.left[node];
    p.pos_right[r] = p.right[node];
  }
  if (!barrier()) return;
  TL_STAMP(trace, kTraceLevels - 1, 2);   // tokens marked
  // (the CTA's operand buffers are idle in this phase: they hold the scan's ballots)
  unsigned int* const s_mask = reinterpret_cast<unsigned int*>(s_dyn4);
  const int mask_cap = (int)(sizeof(BwdSmem) / sizeof(unsigned int));
  int* const group_count = p.tok_slot + p.vocab + 4;   // behind the table and its spare entries
  if (gridDim.x == 1) {
    scan_tokens(p, s_mask, mask_cap);
    classifier_groups(p, 0, 1, s_cls);
  } else {
    scan_count_groups(p, group_count);
    classifier_groups(p, blockIdx.x, gridDim.x, s_cls);
  }
  TL_STAMP(trace, kTraceLevels - 1, 3);   // this CTA's part (the first one: the token scan) done
  if (!barrier()) return;
  TL_STAMP(trace, kTraceLevels - 1, 4);   // classifier, loss and token scan done everywhere
  if (gridDim.x > 1) scan_place_groups(p, group_count);   // needs nothing but the counts; its results are read after the kernel
  // the first wavefront boundaries in shared memory: no dependent global load after every barrier
  // (filled here, ordered before its first use by the CTA barriers inside the grid barrier above)
  constexpr int kOffCache = 256;
  __shared__ int s_off[kOffCache];
  for (int i = threadIdx.x; i < kOffCache && i <= n_levels; i += blockDim.x) s_off[i] = level_offset[i];
  __syncthreads();
  auto level_begin = [&](int l) { return l < kOffCache ? s_off[l] : level_offset[l]; };
  auto is_fused = [&](int l) { return l > 0 && level_begin(l + 1) - level_begin(l) <= kFusedMaxRows; };
  // this CTA's first block of every narrow wavefront, worked out once (thread l: wavefront l) - the
  // divisions behind it would otherwise sit between a wavefront's last store and the grid barrier
  auto first_block = [&](int l) {
    FusedItem it{};   // c_lo == chunks == 0: no block
    if (is_fused(l)) {
      const int b = level_begin(l), e = level_begin(l + 1);
      const int ntiles = dinput_tiles(e - b, 2 * H), nsplits = dinput_splits(ntiles, J);
      if ((int)blockIdx.x < ntiles * nsplits) it = fused_item(p, b, e, blockIdx.x % ntiles, blockIdx.x / ntiles, nsplits);
    }
    return it;
  };
  __shared__ FusedItem s_first[kOffCache];
  for (int l = threadIdx.x; l < kOffCache && l < n_levels; l += blockDim.x) s_first[l] = first_block(l);
  __syncthreads();
  bool prepared = false;
  FusedItem pre_item{};
  FusedFetch pre_fetch;
  for (int lvl = n_levels - 1; lvl >= 0; --lvl) {
    const int begin = level_begin(lvl), end = level_begin(lvl + 1), leaf = lvl == 0 ? 1 : 0;
    const long long elems = (long long)(end - begin) * H;
    TL_STAMP(trace, lvl, 0);
    // a narrow internal wavefront forms its gate gradients inside the contraction (dinput_fused)
    const bool fused = is_fused(lvl);
    if (!fused) {
      for (long long idx = (long long)gtid; idx < elems; idx += (long long)gthreads) gates_element(p, begin, idx, leaf);
      TL_STAMP(trace, lvl, 1);
      if (leaf && !with_dweight) break;   // the leaves' input gradients are left to the tensor-core kernel as well
      if (!barrier()) return;
    }
    TL_STAMP(trace, lvl, 2);
    const int tiles = dinput_tiles(end - begin, leaf ? E : 2 * H), splits = dinput_splits(tiles, J);
    // This CTA's first block of the next wavefront: its index triples and first weight chunk are requested
    // as soon as the operand buffers are free - ahead of the atomic adds of this wavefront's results, which
    // would otherwise hold the requests up - and land in shared memory during the grid barrier.
    bool requested = false;
    auto request_next = [&]() {
      TL_STAMP(trace, lvl, 9);
      requested = true;
      prepared = false;
      if (lvl > 1) {
        pre_item = lvl - 1 < kOffCache ? s_first[lvl - 1] : first_block(lvl - 1);
        if (pre_item.c_lo < pre_item.chunks) {
          fused_fetch(p, pre_item, pre_item.c_lo * BK, pre_fetch);
          prepared = true;
        }
      }
      TL_STAMP(trace, lvl, 11);
    };
    if (fused) {
      for (int vb = blockIdx.x; vb < tiles * splits; vb += gridDim.x) {
        const bool ready = prepared && vb == (int)blockIdx.x;
        const bool last = vb + (int)gridDim.x >= tiles * splits;
        const FusedItem item = ready ? pre_item : fused_item(p, begin, end, vb % tiles, vb / tiles, splits);
        if (last) dinput_fused(p, item, sm.di, lvl & 1, ready, pre_fetch, TL_TRACE_ARG, lvl, request_next);
        else dinput_fused(p, item, sm.di, lvl & 1, ready, pre_fetch, TL_TRACE_ARG, lvl, []() {});
      }
      TL_STAMP(trace, lvl, 7);   // own blocks done
    } else {
      for (int vb = blockIdx.x; vb < tiles * splits; vb += gridDim.x)
        dinput_block(p, begin, end, leaf, vb % tiles, vb / tiles, splits, sm.di);
    }
    if (!requested) request_next();
    TL_STAMP(trace, lvl, 3);
    if (lvl > 0 && !barrier()) return;   // the leaves' dIn goes to the embedding rows only
    TL_STAMP(trace, lvl, 4);
  }
  TL_STAMP(trace, kTraceLevels - 1, 5);   // all wavefronts done
  if (!with_dweight) return;              // dW, db and the leaves' dIn are left to the tensor-core kernel that follows on the stream
  const int tiles_j = (J + BT - 1) / BT, rows_per_split = kDwRows;
  for (int part = 0; part < 2; ++part) {
    const int begin = part == 0 ? 0 : p.n_leaves, end = part == 0 ? p.n_leaves : n;
    if (end <= begin) continue;
    const int K = part == 0 ? E : 2 * H;
    const int nbx = ((K + BT - 1) / BT) * tiles_j, nby = (end - begin + rows_per_split - 1) / rows_per_split;
    for (int vb = blockIdx.x; vb < nbx * nby; vb += gridDim.x)
      dweight_block(p, part, begin, end, rows_per_split, vb % nbx, vb / nbx, sm.dw);
    TL_STAMP(trace, kTraceLevels - 1, 6 + part);   // this CTA's blocks of dW from the leaves / the internal nodes done
  }
  const int nby = (n + 255) / 256;
  for (long long idx = (long long)gtid; idx < (long long)J * nby; idx += (long long)gthreads)
    dbias_piece(p, (int)(idx % J), (int)(idx / J));
  TL_STAMP(trace, kTraceLevels - 1, 8);
}

}  // namespace

int launch_backward(treelstm* ctx, const int32_t* labels, float* loss, float* dW, float* db,
                    float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows,
                    int32_t* n_touched, cudaStream_t stream) {
  auto& L = ctx->last;
  L.stream = stream;
  const bool one_launch = !L.host_levels_valid;   // the forward kept the level table on the device
  if (!one_launch) {
    int rc = ensure_host_levels(ctx);
    if (rc != TREELSTM_OK) return rc;
  }
  const int n = L.n, H = ctx->H, E = ctx->E, C = ctx->C, n_levels = one_launch ? 0 : L.n_levels;
  const int32_t* off = ctx->host_level_offset;
  char* base = static_cast<char*>(L.ws);
  BwdParams p;
  p.n = n; p.H = H; p.E = E; p.C = C; p.vocab = ctx->vocab;
  p.n_leaves = n_levels > 0 ? off[1] : 0;
  p.left = L.left; p.right = L.right; p.token = L.token; p.order = L.order; p.labels = labels;
  p.emb = ctx->emb; p.W = ctx->W; p.Wc = ctx->Wc; p.bc = ctx->bc; p.h = L.h; p.c = L.c;
  p.gates = reinterpret_cast<const float*>(base + L.lay.gates);
  p.dh = reinterpret_cast<float*>(base + L.lay.dh);
  p.dc = reinterpret_cast<float*>(base + L.lay.dc);
  p.dz = reinterpret_cast<float*>(base + L.lay.dz);
  p.loss = loss; p.dW = dW; p.db = db; p.dWc = dWc; p.dbc = dbc; p.dEmb_rows = dEmb_rows;
  p.tok_slot = reinterpret_cast<int*>(base + L.lay.tok_slot);
  p.touched_ids = touched_ids; p.n_touched = n_touched;
  p.pos_left = reinterpret_cast<int*>(base + L.lay.parent);      // the scheduler's scratch is free once the forward has run
  p.pos_right = reinterpret_cast<int*>(base + L.lay.order_tmp);
  p.st = reinterpret_cast<DevStatus*>(base + L.lay.status);
  p.trace = nullptr;
#ifdef TREELSTM_TRACE
  p.trace = reinterpret_cast<long long*>(base + L.lay.trace);   // the forward's table: an fp32 forward leaves it unused
  TL_CUDA(ctx, cudaMemsetAsync(p.trace, 0, sizeof(long long) * kTraceSlots * kTraceLevels, stream));
#endif

  const size_t J = 5 * (size_t)H;
  const size_t cls_smem = sizeof(float) * ((size_t)H * C + C);
  if (cls_smem > 160 * 1024) return TREELSTM_ERR_UNSUPPORTED;
  if (one_launch) {
    if (n == 0) {
      TL_CUDA(ctx, cudaMemsetAsync(loss, 0, sizeof(float), stream));
      TL_CUDA(ctx, cudaMemsetAsync(dW, 0, sizeof(float) * (E + 2 * (size_t)H) * J, stream));
      TL_CUDA(ctx, cudaMemsetAsync(db, 0, sizeof(float) * J, stream));
      TL_CUDA(ctx, cudaMemsetAsync(dWc, 0, sizeof(float) * H * C, stream));
      TL_CUDA(ctx, cudaMemsetAsync(dbc, 0, sizeof(float) * C, stream));
      TL_CUDA(ctx, cudaMemsetAsync(n_touched, 0, sizeof(int), stream));
      return TREELSTM_OK;
    }
    const size_t smem = ((sizeof(BwdSmem) + 3) / 4) * 4 + cls_smem;
    TL_CUDA(ctx, cudaFuncSetAttribute(k_bwd_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    TL_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_bwd_persistent, 256, smem));
    if (per_sm < 1) return TREELSTM_ERR_UNSUPPORTED;
    int grid = ctx->sm_count * (per_sm < 2 ? per_sm : 2);
    if (ctx->opt.max_ctas > 0 && grid > ctx->opt.max_ctas) grid = ctx->opt.max_ctas;
    DevStatus* st = p.st;
    TL_CUDA(ctx, cudaMemsetAsync(&st->barrier_bwd, 0, sizeof(unsigned int), stream));
    const int* lvl_off = L.level_offset;
    long long wait_limit = ctx->opt.wait_limit_kcycles * 1024;
    int with_dweight = ctx->opt.dw_tensor_cores ? 0 : 1;
    void* args[] = {&p, &lvl_off, &wait_limit, &with_dweight};
    TL_CUDA(ctx, cudaLaunchCooperativeKernel((void*)k_bwd_persistent, dim3(grid), dim3(256), args, smem, stream));
    ctx->launches += 1;
    if (!with_dweight)
      return launch_dweight_tc(ctx, n, L.order, L.level_offset, L.token, L.left, L.right, L.h, p.dz, dW, db, p.tok_slot,
                               dEmb_rows, p.st, stream);
    return TREELSTM_OK;
  }
  TL_CUDA(ctx, cudaMemsetAsync(loss, 0, sizeof(float), stream));
  TL_CUDA(ctx, cudaMemsetAsync(dW, 0, sizeof(float) * (E + 2 * (size_t)H) * J, stream));
  TL_CUDA(ctx, cudaMemsetAsync(db, 0, sizeof(float) * J, stream));
  TL_CUDA(ctx, cudaMemsetAsync(dWc, 0, sizeof(float) * H * C, stream));
  TL_CUDA(ctx, cudaMemsetAsync(dbc, 0, sizeof(float) * C, stream));
  TL_CUDA(ctx, cudaMemsetAsync(n_touched, 0, sizeof(int), stream));
  if (n == 0) return TREELSTM_OK;
  TL_CUDA(ctx, cudaMemsetAsync(p.dc, 0, sizeof(float) * (size_t)n * H, stream));
  TL_CUDA(ctx, cudaMemsetAsync(p.tok_slot, 0, sizeof(int) * ((size_t)ctx->vocab + 1), stream));
  TL_CUDA(ctx, cudaMemsetAsync(dEmb_rows, 0, sizeof(float) * (size_t)p.n_leaves * E, stream));

  k_bwd_mark_tokens<<<(p.n_leaves + 255) / 256, 256, 0, stream>>>(p);
  k_bwd_scan_tokens<<<1, 1024, 0, stream>>>(p);
  if (cls_smem > 48 * 1024)
    TL_CUDA(ctx, cudaFuncSetAttribute(k_bwd_classifier, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)cls_smem));
  k_bwd_classifier<<<(n + kClsNodesPerCta - 1) / kClsNodesPerCta, kClsWarps * 32, cls_smem, stream>>>(p);
  ctx->launches += 3;
  for (int lvl = n_levels - 1; lvl >= 0; --lvl) {
    const int begin = off[lvl], end = off[lvl + 1], leaf = lvl == 0 ? 1 : 0;
    const long long elems = (long long)(end - begin) * H;
    k_bwd_gates<<<(unsigned)((elems + 255) / 256), 256, 0, stream>>>(p, begin, end, leaf);
    const int tiles = dinput_tiles(end - begin, leaf ? E : 2 * H), splits = dinput_splits(tiles, (int)J);
    k_bwd_dinput<<<dim3(tiles, splits), 256, 0, stream>>>(p, begin, end, leaf);
    ctx->launches += 2;
  }
  const int tiles_j = (int)((J + BT - 1) / BT);
  for (int part = 0; part < 2; ++part) {
    const int begin = part == 0 ? 0 : p.n_leaves, end = part == 0 ? p.n_leaves : n;
    if (end <= begin) continue;
    const int K = part == 0 ? E : 2 * H;
    const int rows_per_split = kDwRows;
    const int splits = (end - begin + rows_per_split - 1) / rows_per_split;
    dim3 grid(((K + BT - 1) / BT) * tiles_j, splits);
    k_bwd_dweight<<<grid, 256, 0, stream>>>(p, part, begin, end, rows_per_split);
    ctx->launches += 1;
  }
  dim3 gb((unsigned)((J + 127) / 128), (n + 255) / 256);
  k_bwd_dbias<<<gb, 128, 0, stream>>>(p);
  ctx->launches += 1;
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}


// ---- TreeRNN / RNTN: backward through structure ------------------------------------------------ //
// Section 4.2.2 for the two other evaluation models of Section 6.1, on the same schedule.  An
// internal node n with x = [h_l ; h_r], p = h_n = tanh(z):
//     dz   = dh_n * (1 - p^2)
//     dW  += x (x) dz,  db += dz,  RNTN: dV_j += dz_j * x (x) x
//     dx   = W dz  (+ RNTN: sum_j dz_j (V_j + V_j^T) x)      -> added to dh of the two children
// a leaf's state is its word vector: dEmb[token] += dh.  Wavefronts in reverse, one launch per phase
// and wavefront; plain fp32, one thread per output element - correct and measured, not tuned.
namespace {

struct RecBwd {
  int n, H, n_leaves, tensor;
  const int *left, *right, *token, *order;
  const float *h, *W, *Vt;     // W [2H][H]; Vt [(a * 2H + b)][j] = V[j][a][b]
  float *dh, *dz;
  float *dW, *db, *dV, *dEmb_rows;
  const int* tok_slot;
  DevStatus* st;
};

__global__ void k_rec_bwd_dz(RecBwd p, int begin, int end) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)(end - begin) * p.H) return;
  const int node = chk(p.st, p.order[begin + (int)(idx / p.H)], p.n), u = (int)(idx % p.H);
  const float hv = p.h[(size_t)node * p.H + u];
  p.dz[(size_t)node * p.H + u] = p.dh[(size_t)node * p.H + u] * (1.f - hv * hv);
}

// one thread per (node of the wavefront, input unit a in [0, 2H)); a child has one caller, so its dh
// is updated without atomics
__global__ void k_rec_bwd_dx(RecBwd p, int begin, int end) {
  const int H = p.H, K = 2 * H;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)(end - begin) * K) return;
  const int node = chk(p.st, p.order[begin + (int)(idx / K)], p.n), a = (int)(idx % K);
  const int l = chk(p.st, p.left[node], p.n), r = chk(p.st, p.right[node], p.n);
  const float* dz = p.dz + (size_t)node * H;
  float acc = 0.f;
  for (int j = 0; j < H; ++j) acc = fmaf(p.W[(size_t)a * H + j], dz[j], acc);
  if (p.tensor) {
    const float* hl = p.h + (size_t)l * H;
    const float* hr = p.h + (size_t)r * H;
    for (int b = 0; b < K; ++b) {
      const float xb = b < H ? hl[b] : hr[b - H];
      const float* vab = p.Vt + ((size_t)a * K + b) * H;
      const float* vba = p.Vt + ((size_t)b * K + a) * H;
      float t = 0.f;
      for (int j = 0; j < H; ++j) t = fmaf(dz[j], vab[j] + vba[j], t);
      acc = fmaf(t, xb, acc);
    }
  }
  const int child = a < H ? l : r;
  p.dh[(size_t)child * H + (a < H ? a : a - H)] += acc;
}

__global__ void k_rec_bwd_leaves(RecBwd p) {
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)p.n_leaves * p.H) return;
  const int node = chk(p.st, p.order[(int)(idx / p.H)], p.n), u = (int)(idx % p.H);
  const int row = p.tok_slot[p.token[node]];
  atomicAdd(&p.dEmb_rows[(size_t)row * p.H + u], p.dh[(size_t)node * p.H + u]);
}

// one thread per element of dW [2H][H] (+ db [H] in the threads of row 0): a fixed order of summation
__global__ void k_rec_bwd_dw(RecBwd p) {
  const int H = p.H, K = 2 * H;
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= K * H) return;
  const int a = idx / H, j = idx % H;
  float acc = 0.f, accb = 0.f;
  for (int pos = p.n_leaves; pos < p.n; ++pos) {
    const int node = p.order[pos];
    const int child = a < H ? p.left[node] : p.right[node];
    const float dzj = p.dz[(size_t)node * H + j];
    acc = fmaf(p.h[(size_t)child * H + (a < H ? a : a - H)], dzj, acc);
    accb += dzj;
  }
  p.dW[idx] = acc;
  if (a == 0) p.db[j] = accb;
}

// one thread per element of dV [H][2H][2H]
__global__ void k_rec_bwd_dv(RecBwd p) {
  const int H = p.H, K = 2 * H;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)H * K * K) return;
  const int j = (int)(idx / ((long long)K * K)), a = (int)((idx / K) % K), b = (int)(idx % K);
  float acc = 0.f;
  for (int pos = p.n_leaves; pos < p.n; ++pos) {
    const int node = p.order[pos];
    const int l = p.left[node], r = p.right[node];
    const float xa = a < H ? p.h[(size_t)l * H + a] : p.h[(size_t)r * H + a - H];
    const float xb = b < H ? p.h[(size_t)l * H + b] : p.h[(size_t)r * H + b - H];
    acc = fmaf(p.dz[(size_t)node * H + j], xa * xb, acc);
  }
  p.dV[idx] = acc;
}

}  // namespace

int launch_backward_rec(treelstm* ctx, const int32_t* labels, float* loss, float* dW, float* db, float* dV,
                        float* dWc, float* dbc, int32_t* touched_ids, float* dEmb_rows, int32_t* n_touched,
                        cudaStream_t stream) {
  auto& L = ctx->last;
  L.stream = stream;
  int rc = ensure_host_levels(ctx);      // one read of the level table (a persistent forward left it on the device)
  if (rc != TREELSTM_OK) return rc;
  const int n = L.n, H = ctx->H, C = ctx->C, n_levels = L.n_levels;
  const bool tensor = ctx->cell == TREELSTM_CELL_RNTN;
  const int32_t* off = ctx->host_level_offset;
  const size_t K = 2 * (size_t)H;
  TL_CUDA(ctx, cudaMemsetAsync(loss, 0, sizeof(float), stream));
  TL_CUDA(ctx, cudaMemsetAsync(dW, 0, sizeof(float) * K * H, stream));
  TL_CUDA(ctx, cudaMemsetAsync(db, 0, sizeof(float) * H, stream));
  if (tensor) TL_CUDA(ctx, cudaMemsetAsync(dV, 0, sizeof(float) * H * K * K, stream));
  TL_CUDA(ctx, cudaMemsetAsync(dWc, 0, sizeof(float) * H * C, stream));
  TL_CUDA(ctx, cudaMemsetAsync(dbc, 0, sizeof(float) * C, stream));
  TL_CUDA(ctx, cudaMemsetAsync(n_touched, 0, sizeof(int), stream));
  if (n == 0 || n_levels == 0) return TREELSTM_OK;
  char* base = static_cast<char*>(L.ws);
  const int n_leaves = off[1];
  // the classifier, the loss and the touched-token bookkeeping are the TreeLSTM path's kernels
  BwdParams p{};
  p.n = n; p.H = H; p.E = H; p.C = C; p.vocab = ctx->vocab; p.n_leaves = n_leaves;
  p.left = L.left; p.right = L.right; p.token = L.token; p.order = L.order; p.labels = labels;
  p.Wc = ctx->Wc; p.bc = ctx->bc; p.h = L.h;
  p.dh = reinterpret_cast<float*>(base + L.lay.dh);
  p.dz = reinterpret_cast<float*>(base + L.lay.dz);
  p.loss = loss; p.dWc = dWc; p.dbc = dbc; p.dEmb_rows = dEmb_rows;
  p.tok_slot = reinterpret_cast<int*>(base + L.lay.tok_slot);
  p.touched_ids = touched_ids; p.n_touched = n_touched;
  p.st = reinterpret_cast<DevStatus*>(base + L.lay.status);
  const size_t cls_smem = sizeof(float) * ((size_t)H * C + C);
  if (cls_smem > 160 * 1024) return TREELSTM_ERR_UNSUPPORTED;
  TL_CUDA(ctx, cudaMemsetAsync(p.tok_slot, 0, sizeof(int) * ((size_t)ctx->vocab + 1), stream));
  TL_CUDA(ctx, cudaMemsetAsync(dEmb_rows, 0, sizeof(float) * (size_t)n_leaves * H, stream));
  k_bwd_mark_tokens<<<(n_leaves + 255) / 256, 256, 0, stream>>>(p);
  k_bwd_scan_tokens<<<1, 1024, 0, stream>>>(p);
  if (cls_smem > 48 * 1024)
    TL_CUDA(ctx, cudaFuncSetAttribute(k_bwd_classifier, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cls_smem));
  k_bwd_classifier<<<(n + kClsNodesPerCta - 1) / kClsNodesPerCta, kClsWarps * 32, cls_smem, stream>>>(p);
  ctx->launches += 3;

  RecBwd q{};
  q.n = n; q.H = H; q.n_leaves = n_leaves; q.tensor = tensor ? 1 : 0;
  q.left = L.left; q.right = L.right; q.token = L.token; q.order = L.order;
  q.h = L.h; q.Vt = ctx->Wcat; q.W = ctx->Wcat + (tensor ? K * K * H : 0);
  q.dh = p.dh; q.dz = p.dz; q.dW = dW; q.db = db; q.dV = dV; q.dEmb_rows = dEmb_rows; q.tok_slot = p.tok_slot; q.st = p.st;
  for (int lvl = n_levels - 1; lvl >= 1; --lvl) {
    const int begin = off[lvl], end = off[lvl + 1];
    const long long e1 = (long long)(end - begin) * H, e2 = (long long)(end - begin) * (long long)K;
    k_rec_bwd_dz<<<(unsigned)((e1 + 255) / 256), 256, 0, stream>>>(q, begin, end);
    k_rec_bwd_dx<<<(unsigned)((e2 + 127) / 128), 128, 0, stream>>>(q, begin, end);
    ctx->launches += 2;
  }
  k_rec_bwd_leaves<<<(unsigned)(((long long)n_leaves * H + 255) / 256), 256, 0, stream>>>(q);
  ctx->launches += 1;
  if (n > n_leaves) {
    k_rec_bwd_dw<<<(unsigned)((K * H + 127) / 128), 128, 0, stream>>>(q);
    ctx->launches += 1;
    if (tensor) {
      k_rec_bwd_dv<<<(unsigned)((H * K * K + 127) / 128), 128, 0, stream>>>(q);
      ctx->launches += 1;
    }
  }
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

}  // namespace tl
