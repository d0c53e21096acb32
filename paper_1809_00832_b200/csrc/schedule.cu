// On-device ready-set construction for a forest given as child-index arrays.
//
// Paper, Section 4.1.1: an operation with no unresolved input is ready; when an operation
// completes, the operations that waited on it and have all inputs resolved become ready.  For a
// tree node this gives wavefront ("level") 0 for leaves and 1 + max(level of children) for
// internal nodes.  Section 4.1.2: every invocation keeps a pointer to its caller -> parent[].
// The ready order reported to the caller is canonical: ascending (level, node id).
//
// Two implementations produce identical arrays:
//   * k_schedule_single: one CTA, dependency words in shared memory, forests up to 32768 nodes;
//   * a multi-CTA path (dependency counters walked up from the leaves, LSD radix sort with
//     per-chunk histograms) for anything larger.
#include "common.cuh"

namespace tl {
namespace {

constexpr int kSingleThreads = 1024;
constexpr int kSingleWarps = kSingleThreads / 32;
// the dependency words share their shared memory with what comes after them: the radix histogram
// (256 x 32 ints) or the per-thread level counts of the few-levels placement (32 x 1024 uint16)
constexpr size_t kSingleScratch = 65536;
constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ unsigned lanemask_lt() {
  unsigned m;
  asm volatile("mov.u32 %0, %%lanemask_lt;" : "=r"(m));
  return m;
}

// Node check shared by both paths.  Returns 0, or the error code.  is_leaf is set for valid nodes.
__device__ __forceinline__ int check_node(int n, int k, int l, int r, const int* token, int vocab,
                                          bool* is_leaf) {
  if (l < 0 && r < 0) {
    *is_leaf = true;
    if (l != -1 || r != -1) return TREELSTM_ERR_INVALID_FOREST;
    int t = token[k];
    if (t < 0 || t >= vocab) return TREELSTM_ERR_TOKEN_OUT_OF_RANGE;
    return 0;
  }
  *is_leaf = false;
  if (l < 0 || r < 0 || l >= n || r >= n || l == r || l == k || r == k)
    return TREELSTM_ERR_INVALID_FOREST;
  return 0;
}

// ------------------------------------------------------------------------------------------ //
// Stable counting pass executed by one CTA of 32 warps over `n` items.
// Item r of the source sequence is src ? src[r] : r.  key(item) in [0, 256).  Items are written
// to dst ordered by key, ties in source order.  hist is shared memory [256][32] ints.
// After the scan step, bin_starts[b] (b < n_bin_starts) receives the position of the first item
// with key b.
// ------------------------------------------------------------------------------------------ //
struct NoPlace {
  __device__ void operator()(int, int) const {}
};

template <class KeyFn, class PlaceFn = NoPlace>
__device__ void block_counting_pass(int n, const int* src, int* dst, KeyFn key, int* hist,
                                    int* scan_tmp, int* bin_starts, int n_bin_starts,
                                    PlaceFn place = NoPlace()) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < kRadixBins * kSingleWarps; i += kSingleThreads) hist[i] = 0;
  __syncthreads();
  int per_warp = (n + kSingleWarps - 1) / kSingleWarps;
  per_warp = (per_warp + 31) & ~31;
  const int begin = min(n, warp * per_warp), end = min(n, begin + per_warp);
  for (int r0 = begin; r0 < end; r0 += 32) {   // one add per distinct key of the 32 items
    const int r = r0 + lane;
    const bool valid = r < end;
    const unsigned act = __ballot_sync(kFull, valid);
    if (valid) {
      const int k = key(src ? src[r] : r);
      const unsigned peers = __match_any_sync(act, k);
      if (lane == __ffs(peers) - 1) hist[k * kSingleWarps + warp] += __popc(peers);
    }
    __syncwarp();
  }
  __syncthreads();
  // exclusive scan of hist in (bin-major, warp-minor) order: 8 consecutive entries per thread
  {
    constexpr int kPer = kRadixBins * kSingleWarps / kSingleThreads;  // 8
    int v[kPer], sum = 0;
#pragma unroll
    for (int j = 0; j < kPer; ++j) { v[j] = hist[tid * kPer + j]; sum += v[j]; }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int t = __shfl_up_sync(kFull, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) scan_tmp[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = scan_tmp[lane], wi = w;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int t = __shfl_up_sync(kFull, wi, d);
        if (lane >= d) wi += t;
      }
      scan_tmp[lane] = wi - w;
    }
    __syncthreads();
    int run = scan_tmp[warp] + incl - sum;
#pragma unroll
    for (int j = 0; j < kPer; ++j) { hist[tid * kPer + j] = run; run += v[j]; }
  }
  __syncthreads();
  for (int b = tid; b < n_bin_starts; b += kSingleThreads) bin_starts[b] = hist[b * kSingleWarps];
  __syncthreads();
  for (int r0 = begin; r0 < end; r0 += 32) {
    const int r = r0 + lane;
    const bool valid = r < end;
    const unsigned act = __ballot_sync(kFull, valid);
    int item = 0, k = 0, base = 0;
    unsigned peers = 0;
    if (valid) {
      item = src ? src[r] : r;
      k = key(item);
      peers = __match_any_sync(act, k);
      base = hist[k * kSingleWarps + warp];
    }
    __syncwarp();
    if (valid && lane == __ffs(peers) - 1) hist[k * kSingleWarps + warp] = base + __popc(peers);
    __syncwarp();
    if (valid) {
      const int pos = base + __popc(peers & lanemask_lt());
      dst[pos] = item;
      place(pos, item);
    }
  }
  __syncthreads();
}

// Ids of the items with flag(item) set, in ascending order, to dst; returns their number to every
// thread.  One CTA of 32 warps; warp w owns a contiguous range of ids.
template <class FlagFn, class PlaceFn = NoPlace>
__device__ int block_compact(int n, int* dst, FlagFn flag, int* scan_tmp, PlaceFn place = NoPlace()) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int per_warp = (n + kSingleWarps - 1) / kSingleWarps;
  per_warp = (per_warp + 31) & ~31;
  const int begin = min(n, warp * per_warp), end = min(n, begin + per_warp);
  int count = 0;
  for (int r0 = begin; r0 < end; r0 += 32) {
    const int r = r0 + lane;
    count += __popc(__ballot_sync(kFull, r < end && flag(r)));
  }
  __syncthreads();
  if (lane == 0) scan_tmp[warp] = count;
  __syncthreads();
  int total = 0, base = 0;
  for (int w2 = 0; w2 < kSingleWarps; ++w2) {
    const int c = scan_tmp[w2];
    if (w2 < warp) base += c;
    total += c;
  }
  for (int r0 = begin; r0 < end; r0 += 32) {
    const int r = r0 + lane;
    const bool f = r < end && flag(r);
    const unsigned m = __ballot_sync(kFull, f);
    if (f) {
      const int idx = base + __popc(m & lanemask_lt());
      dst[idx] = r;
      place(idx, r);
    }
    base += __popc(m);
  }
  __syncthreads();
  return total;
}

// Ready order, wavefront boundaries and roots in one go for forests of at most 32 wavefronts (the
// usual case: depth grows with the logarithm of the sentence length).  One CTA of 1024 threads;
// thread t owns the contiguous ids [t * npt, (t + 1) * npt).  tab[L][t] (uint16, n_levels x 1024: 2 KB of
// shared memory per wavefront) first counts the thread's nodes of level L, then warp L turns row L into its
// exclusive prefix over the threads, and finally thread t hands out positions level_start[L] +
// tab[L][t]++ to its nodes in ascending id - ascending (level, id) overall, with no key matching at
// all.  The positions are scattered into a shared-memory copy of the order (uint16 ids, `staged`) and
// go out to global memory as whole lines afterwards: one SM cannot afford 4-byte stores to n
// different sectors.  Output as the general path: order[], level_offset[0 .. n_levels), roots[] by
// ascending id; returns the number of roots to every thread.  scan_tmp: shared int[32].
__device__ int place_few_levels(int n, int n_levels, const unsigned short* lv16, int* order, int* level_offset,
                                int* roots, unsigned short* tab, unsigned short* staged, int* scan_tmp,
                                int* stamps) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
#ifdef TREELSTM_TRACE
  const long long t_in = clock64();
#define TL_PLACE_STAMP(i) do { if (tid == 0 && stamps) stamps[i] = (int)(clock64() - t_in); } while (0)
#else
  (void)stamps;
#define TL_PLACE_STAMP(i) do { } while (0)
#endif
  __shared__ int s_level_start[32];
  __shared__ int s_root_total;
  const int npt = ((n + kSingleThreads - 1) / kSingleThreads) | 1;   // odd: the threads' ranges start in different banks
  const int k0 = min(n, tid * npt), k1 = min(n, k0 + npt);
  {
    uint4* z = reinterpret_cast<uint4*>(tab);                   // 2 KB = 128 pieces of 16 bytes per wavefront
    for (int i = tid; i < n_levels * kSingleThreads * 2 / 16; i += kSingleThreads) z[i] = make_uint4(0u, 0u, 0u, 0u);
  }
  __syncthreads();
  TL_PLACE_STAMP(0);
  int my_roots = 0;
  for (int k = k0; k < k1; ++k) {
    const unsigned short v = lv16[k];
    tab[(v & 0x7FFF) * kSingleThreads + tid] += 1;
    my_roots += v >> 15;
  }
  __syncthreads();
  TL_PLACE_STAMP(1);
  // row L -> exclusive prefix over the threads (warp L; lane j takes the 32 threads 32 j .. 32 j + 31)
  if (warp < n_levels) {
    unsigned short* row = tab + warp * kSingleThreads + lane * 32;
    unsigned short v[32];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 x = reinterpret_cast<const uint4*>(row)[q];
      const unsigned int w4[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { v[q * 8 + 2 * j] = (unsigned short)(w4[j] & 0xFFFFu); v[q * 8 + 2 * j + 1] = (unsigned short)(w4[j] >> 16); }
    }
    int sum = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) { const int c = v[j]; v[j] = (unsigned short)sum; sum += c; }
    int incl = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(kFull, incl, d);
      if (lane >= d) incl += t;
    }
    const int base = incl - sum;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      unsigned int w4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        w4[j] = (unsigned int)(unsigned short)(v[q * 8 + 2 * j] + base) | ((unsigned int)(unsigned short)(v[q * 8 + 2 * j + 1] + base) << 16);
      reinterpret_cast<uint4*>(row)[q] = make_uint4(w4[0], w4[1], w4[2], w4[3]);
    }
    if (lane == 31) scan_tmp[warp] = incl;                      // nodes of level `warp`
  }
  __syncthreads();
  TL_PLACE_STAMP(2);
  // level starts (warp 0) and the roots' prefix over the threads (all warps, one value per thread)
  if (warp == 0) {
    const int c = lane < n_levels ? scan_tmp[lane] : 0;
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(kFull, incl, d);
      if (lane >= d) incl += t;
    }
    s_level_start[lane] = incl - c;
    if (lane < n_levels) level_offset[lane] = incl - c;
  }
  __syncthreads();
  int rincl = my_roots;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int t = __shfl_up_sync(kFull, rincl, d);
    if (lane >= d) rincl += t;
  }
  if (lane == 31) scan_tmp[warp] = rincl;
  __syncthreads();
  if (warp == 0) {
    const int c = scan_tmp[lane];
    int incl = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int t = __shfl_up_sync(kFull, incl, d);
      if (lane >= d) incl += t;
    }
    scan_tmp[lane] = incl - c;
    if (lane == 31) s_root_total = incl;
  }
  __syncthreads();
  TL_PLACE_STAMP(3);
  int rpos = scan_tmp[warp] + rincl - my_roots;
  for (int k = k0; k < k1; ++k) {
    const unsigned short v = lv16[k];
    const int lv = v & 0x7FFF;
    unsigned short* cell = tab + lv * kSingleThreads + tid;
    const int pos = s_level_start[lv] + *cell;
    *cell += 1;
    staged[pos] = (unsigned short)k;
    if (v >> 15) roots[rpos++] = k;
  }
  __syncthreads();
  TL_PLACE_STAMP(4);
  for (int i = tid; i < n; i += kSingleThreads) order[i] = staged[i];
  return s_root_total;
}

// One CTA schedules the whole forest in shared memory (forests up to 32768 nodes).
//
// Dependency counters, as in Section 4.1.1: every internal node waits for two inputs.  A finished
// child swaps (its level + 1) into its caller's word; the child that finds the word empty was first
// and stops, the one that finds its sibling's entry knows both inputs are resolved, gives the caller
// level 1 + max and goes on upwards.  No global atomics, no grid-wide rounds.
//
// Dynamic shared memory: uint32 w[n] (dependency words; later the sort's scratch, at least 64 KB),
// uint16 par[n] (caller of each node, the return location of Section 4.1.2; later level | root
// flag), uint16 queue[n / 2] (start nodes of the climb), and with n_parts > 0 uint16 lab[n].
//
// n_parts > 0 additionally deals the trees out to n_parts sub-forests (trees are independent,
// Section 2.2): every node learns the root of its tree by pointer jumping over the caller links,
// the t-th root (ascending node id) goes to sub-forest t mod n_parts, and part_order receives the
// node ids by ascending (sub-forest, level, node id) with part_offset[0 .. n_parts] marking where
// each sub-forest starts.  slot[] (if given) is set to -1 for every node.
__global__ void __launch_bounds__(kSingleThreads, 1)
k_schedule_single(int n, const int* __restrict__ left, const int* __restrict__ right,
                  const int* __restrict__ token, int vocab, int* parent, int* level, int* order,
                  int* order_tmp, int* level_offset, int* roots, int* n_levels_out, DevStatus* st,
                  int n_parts, int* part_order, int* part_offset, int* slot, int cache_children) {
  extern __shared__ __align__(16) unsigned char smem[];
  const size_t w_bytes = (size_t)n * 4 > kSingleScratch ? (((size_t)n * 4 + 15) & ~(size_t)15) : kSingleScratch;
  unsigned int* w = reinterpret_cast<unsigned int*>(smem);
  int* hist = reinterpret_cast<int*>(smem);
  unsigned short* par = reinterpret_cast<unsigned short*>(smem + w_bytes);
  unsigned short* lv16 = par;
  unsigned short* queue = par + (((size_t)n + 7) & ~(size_t)7);   // start nodes of the climb, at most n / 2
  unsigned short* lab = reinterpret_cast<unsigned short*>(
      smem + w_bytes + ((((size_t)n * 2) + 15) & ~(size_t)15) + (((size_t)n + 15) & ~(size_t)15));
  // where shared memory allows (no sub-forest labels, forest small enough): both children of every node,
  // packed, so that the second look at them does not go back to global memory
  unsigned int* lr = cache_children ? reinterpret_cast<unsigned int*>(lab) : nullptr;
  __shared__ int scan_tmp[32];
  __shared__ int s_err, s_maxlevel, s_qhead, s_qtail;
  const int tid = threadIdx.x;
  constexpr unsigned short kNoParent = 0xFFFF;
  constexpr unsigned int kDone = 0x80000000u;
  if (tid < (int)(sizeof(DevStatus) / sizeof(int))) reinterpret_cast<int*>(st)[tid] = 0;
#ifdef TREELSTM_TRACE
  // phase stamps of thread 0 (cycles since the start) in the unused words of the control block
  const long long t_start = clock64();
#define TL_SCHED_STAMP(i) do { if (tid == 0) st->pad[i] = (int)(clock64() - t_start); } while (0)
#else
#define TL_SCHED_STAMP(i) do { } while (0)
#endif
  if (tid == 0) { s_err = 0; s_maxlevel = 0; s_qhead = 0; s_qtail = 0; }
  for (int k = tid; k < n; k += kSingleThreads) { w[k] = 0; par[k] = kNoParent; }
  __syncthreads();
  // A kernel launched behind this one as its programmatic dependent may start now.  The part of it
  // that comes before its own wait for this grid reads nothing this grid writes, except that it
  // uses the (now cleared) control block: its barrier counter, and the status word this grid may
  // still set.
  if (tid == 0) {
    __threadfence();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  TL_SCHED_STAMP(0);   // cleared
  // validate; children record their caller; leaves are complete at once (level 0)
  // Node j of this thread is tid + j * 1024 (at most 32 per thread); leaf_bits remembers which are
  // leaves so that later passes need not look at the child arrays again.
  unsigned int leaf_bits = 0;
  for (int j0 = 0; j0 * kSingleThreads + tid < n; j0 += 8) {   // eight nodes per trip: loads first
    int l[8], r[8], t[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int k = tid + (j0 + j) * kSingleThreads;
      l[j] = k < n ? left[k] : -1;
      r[j] = k < n ? right[k] : -1;
      t[j] = k < n ? token[k] : 0;
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int k = tid + (j0 + j) * kSingleThreads;
      if (k >= n) break;
      int err = 0;
      if (l[j] < 0 && r[j] < 0) {
        if (l[j] != -1 || r[j] != -1) err = TREELSTM_ERR_INVALID_FOREST;
        else if (t[j] < 0 || t[j] >= vocab) err = TREELSTM_ERR_TOKEN_OUT_OF_RANGE;
        else { w[k] = kDone; leaf_bits |= 1u << (j0 + j); }
      } else if (l[j] < 0 || r[j] < 0 || l[j] >= n || r[j] >= n || l[j] == r[j] || l[j] == k || r[j] == k) {
        err = TREELSTM_ERR_INVALID_FOREST;
      } else {
        par[l[j]] = (unsigned short)k;
        par[r[j]] = (unsigned short)k;
        if (lr) lr[k] = (unsigned int)l[j] | ((unsigned int)r[j] << 16);
      }
      if (err) atomicMin(&s_err, err);
    }
  }
  __syncthreads();
  TL_SCHED_STAMP(1);   // validated and linked
  if (s_err == 0) {
    // a child claimed by two callers kept only one of them: checked at the caller
    for (int j0 = 0; j0 * kSingleThreads + tid < n; j0 += 8) {
      int l[8], r[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int k = tid + (j0 + j) * kSingleThreads;
        const bool internal = k < n && !((leaf_bits >> (j0 + j)) & 1u);
        if (lr) {
          const unsigned int both = internal ? lr[k] : 0xFFFFFFFFu;
          l[j] = internal ? (int)(both & 0xFFFFu) : -1;
          r[j] = internal ? (int)(both >> 16) : -1;
        } else {
          l[j] = internal ? left[k] : -1;
          r[j] = internal ? right[k] : -1;
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int k = tid + (j0 + j) * kSingleThreads;
        if (l[j] >= 0 && (par[l[j]] != k || par[r[j]] != k)) atomicMin(&s_err, (int)TREELSTM_ERR_INVALID_FOREST);
      }
    }
    // Every leaf reports to its caller.  A caller whose second child reports here is complete
    // (level 1) and goes into the queue of nodes to climb from; climbing starts only after all
    // leaves have reported, so no climb waits for a leaf its owner has not reached yet.
    for (unsigned int bits = leaf_bits; bits; bits &= bits - 1) {
      const int k = tid + (__ffs(bits) - 1) * kSingleThreads;
      const unsigned short p = par[k];
      if (p == kNoParent) continue;
      if (atomicExch(&w[p], 1u) != 0) {         // both children are leaves
        w[p] = kDone | 1u;
        queue[atomicAdd(&s_qtail, 1)] = p;
      }
    }
  }
  __syncthreads();
  TL_SCHED_STAMP(2);   // links checked, leaves reported
  if (s_err == 0) {
    // Climb: threads take start nodes from the queue until it is empty.
    for (;;) {
      const int q = atomicAdd(&s_qhead, 1);
      if (q >= s_qtail) break;
      int cur = queue[q], lvl = 1;
      for (int step = 0; step < n; ++step) {   // a path to the root has fewer than n edges
        const unsigned short p = par[cur];
        if (p == kNoParent) break;
        const unsigned int old = atomicExch(&w[p], (unsigned int)lvl + 1u);
        if (old == 0) break;                   // sibling subtree still unresolved
        lvl = 1 + max(lvl, (int)old - 1);
        w[p] = kDone | (unsigned int)lvl;
        cur = p;
      }
    }
  }
  __syncthreads();
  TL_SCHED_STAMP(3);   // climbed
  int local_max = 0;
  if (s_err == 0) {
    for (int k = tid; k < n; k += kSingleThreads) {
      const unsigned int wk = w[k];
      if (!(wk & kDone)) atomicMin(&s_err, (int)TREELSTM_ERR_INVALID_FOREST);   // on a cycle: never ready
      const int lvl = (int)(wk & 0x7FFFu);
      const unsigned short pk = par[k];
      lv16[k] = (unsigned short)(lvl | (pk == kNoParent ? 0x8000 : 0));
      if (n_parts > 0) {
        lab[k] = pk == kNoParent ? (unsigned short)k : pk;   // start of the pointer jumping
        if (slot) slot[k] = -1;
      }
      level[k] = lvl;
      local_max = max(local_max, lvl);
    }
    atomicMax(&s_maxlevel, local_max);
  }
  __syncthreads();
  if (s_err != 0) {
    if (tid == 0) { report(st, s_err); *n_levels_out = 0; }
    return;
  }
  const int n_levels = n > 0 ? s_maxlevel + 1 : 0;
  TL_SCHED_STAMP(4);   // levels written
  // The few-levels placement needs 2 KB per wavefront for its counts and 2 n bytes for the staged
  // order: the packed children's shared memory (no longer needed) takes the latter, or what the
  // dependency words leave free behind the counts.
  const size_t tab_bytes = (size_t)n_levels * kSingleThreads * 2;
  unsigned short* staged = lr != nullptr ? reinterpret_cast<unsigned short*>(lr)
                           : (tab_bytes + (size_t)n * 2 <= w_bytes ? reinterpret_cast<unsigned short*>(smem + tab_bytes) : nullptr);
  if (n_levels <= 32 && n_parts == 0 && staged != nullptr) {
    const int n_roots = place_few_levels(n, n_levels, lv16, order, level_offset, roots,
                                         reinterpret_cast<unsigned short*>(smem), staged, scan_tmp, st->pad + 8);
    if (tid == 0) {
      level_offset[n_levels] = n; st->n_levels = n_levels; *n_levels_out = n_levels;
      st->n_roots = n_roots;
    }
    TL_SCHED_STAMP(5);   // ordered
    return;
  }
  // canonical ready order: LSD radix on the level, 8 bits per pass, ties by node id
  int passes = 1;
  while (passes < 4 && (n_levels - 1) >> (8 * passes)) ++passes;
  for (int p = 0; p < passes; ++p) {
    int* dst = ((passes - 1 - p) & 1) ? order_tmp : order;
    const int* src = p == 0 ? nullptr : (dst == order ? order_tmp : order);
    const int shift = 8 * p;
    block_counting_pass(n, src, dst, [=](int item) { return ((lv16[item] & 0x7FFF) >> shift) & 255; },
                        hist, scan_tmp, passes == 1 ? level_offset : nullptr, passes == 1 ? n_levels : 0);
  }
  if (passes > 1) {   // wavefront boundaries from the sorted order
    for (int r = tid; r < n; r += kSingleThreads) {
      const int a = lv16[order[r]] & 0x7FFF;
      if (r == 0 || (lv16[order[r - 1]] & 0x7FFF) != a) level_offset[a] = r;
    }
  }
  if (tid == 0) { level_offset[n_levels] = n; st->n_levels = n_levels; *n_levels_out = n_levels; }
  if (n_parts > 0) {
    // lab[k] = root of k's tree: every node replaces its link by its link's link until all links
    // end at a root (a root links to itself); ceil(log2(depth)) + 1 rounds.  Updates are made in
    // place: a link read while it is being advanced is still an ancestor.
    for (int round = 0; round < 17; ++round) {
      int changed = 0;
      for (int k = tid; k < n; k += kSingleThreads) {
        const unsigned short a = lab[k], b = lab[a];
        if (b != a) { lab[k] = b; changed = 1; }
      }
      if (!__syncthreads_or(changed)) break;
    }
  }
  // roots (nodes without a caller) in ascending node id; the t-th root takes sub-forest t mod n_parts
  const int n_roots = block_compact(n, roots, [=](int item) { return (lv16[item] & 0x8000) != 0; }, scan_tmp,
                                    [=](int idx, int item) { if (n_parts > 0) lab[item] = (unsigned short)(idx % n_parts); });
  if (tid == 0) st->n_roots = n_roots;
  if (n_parts > 0) {
    // every other node takes its root's sub-forest (its own entry is read by nobody else: links
    // end at roots only)
    for (int k = tid; k < n; k += kSingleThreads)
      if (!(lv16[k] & 0x8000)) lab[k] = lab[lab[k]];
    __syncthreads();
    // stable pass over the ready order by sub-forest: ascending (sub-forest, level, node id)
    block_counting_pass(n, order, part_order, [=](int item) { return (int)lab[item]; }, hist, scan_tmp,
                        part_offset, n_parts);
    if (tid == 0) part_offset[n_parts] = n;
  }
}

// ------------------------------------------------------------------------------------------ //
// multi-CTA path
// ------------------------------------------------------------------------------------------ //
__global__ void k_sched_init(int n, const int* __restrict__ left, const int* __restrict__ right,
                             const int* __restrict__ token, int vocab, int* parent, int* level,
                             DevStatus* st) {
  // parent[] was set to -1 and pending[] to 0 by memsets enqueued before this kernel
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n) return;
  const int l = left[k], r = right[k];
  bool leaf;
  int err = check_node(n, k, l, r, token, vocab, &leaf);
  if (err == 0 && !leaf) {
    if (atomicCAS(&parent[l], -1, k) != -1) err = TREELSTM_ERR_INVALID_FOREST;
    if (atomicCAS(&parent[r], -1, k) != -1) err = TREELSTM_ERR_INVALID_FOREST;
  }
  if (err) report(st, err);
  level[k] = (err == 0 && leaf) ? 0 : -1;
}

// Dependency counters: every leaf walks towards its root; at each caller the first child to
// arrive stops, the second one knows both children are resolved, assigns the level and goes on.
__global__ void k_sched_walkup(int n, const int* __restrict__ left, const int* __restrict__ right,
                               const int* parent, int* pending, int* level, DevStatus* st) {
  if (ld_volatile(&st->status) != 0) return;
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n || left[k] >= 0) return;
  int cur = k, lvl = 0;
  for (int step = 0; step < n; ++step) {  // a path has fewer than n edges
    const int p = parent[cur];
    if (p < 0) break;
    __threadfence();
    if (atomicAdd(&pending[p], 1) == 0) return;  // sibling subtree still running
    __threadfence();
    const int sib = left[p] == cur ? right[p] : left[p];
    lvl = 1 + max(lvl, ld_volatile(&level[sib]));
    *(volatile int*)&level[p] = lvl;
    cur = p;
  }
  atomicMax(&st->max_level, lvl);
}

__global__ void k_sched_check(int n, const int* level, DevStatus* st) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k == 0 && st->status == 0) st->n_levels = n > 0 ? st->max_level + 1 : 0;
  if (k < n && level[k] < 0) report(st, TREELSTM_ERR_INVALID_FOREST);  // cycle
}

// mode 0: key = digit `pass` of level; mode 1: key = has-a-caller flag.
__device__ __forceinline__ int sort_key(int mode, int pass, int item, const int* level,
                                        const int* parent) {
  return mode == 0 ? ((level[item] >> (8 * pass)) & 255) : (parent[item] >= 0 ? 1 : 0);
}

__device__ __forceinline__ int passes_needed(int n_levels) {
  int passes = 1;
  while (passes < 4 && (n_levels - 1) >> (8 * passes)) ++passes;
  return passes;
}

// Which buffer pass p reads and writes, so that the last needed pass lands in `order`.
__device__ __forceinline__ void pass_buffers(int mode, int pass, int passes, int* order,
                                             int* order_tmp, int* roots, const int** src,
                                             int** dst) {
  if (mode == 1) { *src = nullptr; *dst = roots; return; }
  *dst = ((passes - 1 - pass) & 1) ? order_tmp : order;
  *src = pass == 0 ? nullptr : (*dst == order ? order_tmp : order);
}

// One warp per CTA, chunk of kRadixChunk consecutive source items; table is [256][n_chunks].
__global__ void __launch_bounds__(32)
k_radix_hist(int n, int mode, int pass, const int* level, const int* parent, int* order,
             int* order_tmp, int* roots, int* table, int n_chunks, const DevStatus* st) {
  if (st->status != 0) return;
  const int passes = mode == 0 ? passes_needed(st->n_levels) : 1;
  if (pass >= passes) return;
  __shared__ int hist[kRadixBins];
  const int lane = threadIdx.x, chunk = blockIdx.x;
  for (int i = lane; i < kRadixBins; i += 32) hist[i] = 0;
  __syncwarp();
  const int* src; int* dst;
  pass_buffers(mode, pass, passes, order, order_tmp, roots, &src, &dst);
  const int begin = chunk * kRadixChunk, end = min(n, begin + kRadixChunk);
  for (int r = begin + lane; r < end; r += 32) {
    const int item = src ? src[r] : r;
    atomicAdd(&hist[sort_key(mode, pass, item, level, parent)], 1);
  }
  __syncwarp();
  for (int i = lane; i < kRadixBins; i += 32) table[(size_t)i * n_chunks + chunk] = hist[i];
}

// Exclusive scan of the whole table by one CTA.
__global__ void __launch_bounds__(1024)
k_radix_scan(int mode, int pass, int* table, int n_chunks, DevStatus* st) {
  if (st->status != 0) return;
  const int passes = mode == 0 ? passes_needed(st->n_levels) : 1;
  if (pass >= passes) return;
  __shared__ int warp_sum[32];
  __shared__ int carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long total = (long long)kRadixBins * n_chunks;
  if (tid == 0) carry = 0;
  __syncthreads();
  for (long long base = 0; base < total; base += 1024) {
    const long long i = base + tid;
    const int v = i < total ? table[i] : 0;
    int incl = v;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int t = __shfl_up_sync(kFull, incl, d);
      if (lane >= d) incl += t;
    }
    if (lane == 31) warp_sum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int w = warp_sum[lane], wi = w;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        int t = __shfl_up_sync(kFull, wi, d);
        if (lane >= d) wi += t;
      }
      warp_sum[lane] = wi - w;
    }
    __syncthreads();
    const int excl = carry + warp_sum[warp] + incl - v;
    if (i < total) table[i] = excl;
    if (mode == 1 && i == (long long)n_chunks) st->n_roots = excl;  // start of bin 1
    __syncthreads();
    if (tid == 1023) carry = excl + v;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(32)
k_radix_scatter(int n, int mode, int pass, const int* level, const int* parent, int* order,
                int* order_tmp, int* roots, const int* table, int n_chunks, const DevStatus* st) {
  if (st->status != 0) return;
  const int passes = mode == 0 ? passes_needed(st->n_levels) : 1;
  if (pass >= passes) return;
  __shared__ int base_of[kRadixBins];
  const int lane = threadIdx.x, chunk = blockIdx.x;
  for (int i = lane; i < kRadixBins; i += 32) base_of[i] = table[(size_t)i * n_chunks + chunk];
  __syncwarp();
  const int* src; int* dst;
  pass_buffers(mode, pass, passes, order, order_tmp, roots, &src, &dst);
  const int begin = chunk * kRadixChunk, end = min(n, begin + kRadixChunk);
  for (int r0 = begin; r0 < end; r0 += 32) {
    const int r = r0 + lane;
    const bool valid = r < end;
    const unsigned act = __ballot_sync(kFull, valid);
    int item = 0, k = 0, base = 0;
    unsigned peers = 0;
    if (valid) {
      item = src ? src[r] : r;
      k = sort_key(mode, pass, item, level, parent);
      peers = __match_any_sync(act, k);
      base = base_of[k];
    }
    __syncwarp();
    if (valid && lane == __ffs(peers) - 1) base_of[k] = base + __popc(peers);
    __syncwarp();
    if (valid) dst[base + __popc(peers & lanemask_lt())] = item;
  }
}

__global__ void k_sched_offsets(int n, const int* level, const int* order, int* level_offset,
                                const DevStatus* st) {
  if (st->status != 0) return;
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r == 0) level_offset[st->n_levels] = n;
  if (r >= n) return;
  const int a = level[order[r]];
  if (r == 0 || level[order[r - 1]] != a) level_offset[a] = r;
}

__global__ void k_gather_roots(int max_roots, int H, const int* roots, const float* h,
                               const float* c, int* root_ids, float* root_h, float* root_c,
                               int* n_roots_out, const DevStatus* st) {
  const int n_roots = st->status == 0 ? min(st->n_roots, max_roots) : 0;
  if (blockIdx.x == 0 && threadIdx.x == 0 && n_roots_out) *n_roots_out = n_roots;
  for (int t = blockIdx.x; t < n_roots; t += gridDim.x) {
    const int node = roots[t];   // written by the scheduler from ids below n
    if (threadIdx.x == 0 && root_ids) root_ids[t] = node;
    for (int j = threadIdx.x; j < H; j += blockDim.x) {
      if (root_h) root_h[(size_t)t * H + j] = h[(size_t)node * H + j];
      if (root_c) root_c[(size_t)t * H + j] = c[(size_t)node * H + j];
    }
  }
}

}  // namespace

size_t single_smem_bytes(int n, bool with_parts) {
  size_t w = (size_t)n * 4;
  w = w > kSingleScratch ? round_up_sz(w, 16) : kSingleScratch;
  return w + round_up_sz((size_t)n * 2, 16) + round_up_sz((size_t)n, 16) +
         (with_parts ? round_up_sz((size_t)n * 2, 16) : 0);
}
// The packed children of every node next to the rest, if that still fits one CTA's shared memory.
bool single_caches_children(int n, bool with_parts) {
  return !with_parts && single_smem_bytes(n, false) + (size_t)n * 4 + 16 <= single_smem_bytes(kSchedSingleMaxNodes, false);
}

int init_schedule_attributes(treelstm* ctx) {
  TL_CUDA(ctx, cudaFuncSetAttribute(k_schedule_single, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)single_smem_bytes(kSchedSingleMaxNodes, false)));
  return TREELSTM_OK;
}

int launch_schedule(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                    const int32_t* token, int32_t* level, int32_t* order, int32_t* level_offset,
                    int32_t* n_levels_out, void* ws, const WsLayout& lay, int n_parts, cudaStream_t stream) {
  char* base = static_cast<char*>(ws);
  DevStatus* st = reinterpret_cast<DevStatus*>(base + lay.status);
  int* parent = reinterpret_cast<int*>(base + lay.parent);
  int* pending = reinterpret_cast<int*>(base + lay.pending);
  int* order_tmp = reinterpret_cast<int*>(base + lay.order_tmp);
  int* roots = reinterpret_cast<int*>(base + lay.roots);
  int* table = reinterpret_cast<int*>(base + lay.table);

  const int single_max = ctx->opt.sched_single_cta_max < kSchedSingleMaxNodes
                             ? ctx->opt.sched_single_cta_max : kSchedSingleMaxNodes;
  if (n > 0 && n <= single_max) {
    // the kernel clears the control block itself and writes the level count to the caller
    const bool parts = n_parts > 0 && n <= kSchedPartMaxNodes;
    const bool cache = single_caches_children(n, parts);
    k_schedule_single<<<1, kSingleThreads, single_smem_bytes(n, parts) + (cache ? (size_t)n * 4 + 16 : 0), stream>>>(
        n, left, right, token, ctx->vocab, parent, level, order, order_tmp, level_offset, roots, n_levels_out,
        st, parts ? n_parts : 0, reinterpret_cast<int*>(base + lay.part_order),
        reinterpret_cast<int*>(base + lay.part_offset), reinterpret_cast<int*>(base + lay.slot), cache ? 1 : 0);
    ctx->launches += 1;
    TL_CUDA(ctx, cudaGetLastError());
    return TREELSTM_OK;
  }

  TL_CUDA(ctx, cudaMemsetAsync(st, 0, sizeof(DevStatus), stream));
  if (n == 0) {
    TL_CUDA(ctx, cudaMemsetAsync(n_levels_out, 0, sizeof(int), stream));
    return TREELSTM_OK;
  }
  TL_CUDA(ctx, cudaMemsetAsync(parent, 0xFF, sizeof(int) * (size_t)n, stream));
  TL_CUDA(ctx, cudaMemsetAsync(pending, 0, sizeof(int) * (size_t)n, stream));
  const int tpb = 256, blocks = (n + tpb - 1) / tpb;
  k_sched_init<<<blocks, tpb, 0, stream>>>(n, left, right, token, ctx->vocab, parent, level, st);
  k_sched_walkup<<<blocks, tpb, 0, stream>>>(n, left, right, parent, pending, level, st);
  k_sched_check<<<blocks, tpb, 0, stream>>>(n, level, st);
  ctx->launches += 3;
  const int n_chunks = (n + kRadixChunk - 1) / kRadixChunk;
  // a forest of n nodes has at most (n + 1) / 2 levels; later passes switch themselves off on
  // the device once the actual level count is known
  int host_passes = 1;
  while (host_passes < 4 && (((n + 1) / 2 - 1) >> (8 * host_passes))) ++host_passes;
  for (int p = 0; p < host_passes; ++p) {
    k_radix_hist<<<n_chunks, 32, 0, stream>>>(n, 0, p, level, parent, order, order_tmp, roots, table,
                                              n_chunks, st);
    k_radix_scan<<<1, 1024, 0, stream>>>(0, p, table, n_chunks, st);
    k_radix_scatter<<<n_chunks, 32, 0, stream>>>(n, 0, p, level, parent, order, order_tmp, roots,
                                                 table, n_chunks, st);
    ctx->launches += 3;
  }
  k_sched_offsets<<<blocks, tpb, 0, stream>>>(n, level, order, level_offset, st);
  k_radix_hist<<<n_chunks, 32, 0, stream>>>(n, 1, 0, level, parent, order, order_tmp, roots, table,
                                            n_chunks, st);
  k_radix_scan<<<1, 1024, 0, stream>>>(1, 0, table, n_chunks, st);
  k_radix_scatter<<<n_chunks, 32, 0, stream>>>(n, 1, 0, level, parent, order, order_tmp, roots,
                                               table, n_chunks, st);
  ctx->launches += 4;
  TL_CUDA(ctx, cudaGetLastError());
  TL_CUDA(ctx, cudaMemcpyAsync(n_levels_out, &st->n_levels, sizeof(int), cudaMemcpyDeviceToDevice, stream));
  return TREELSTM_OK;
}

#ifdef TREELSTM_CHECKED
namespace {
// After a forward: every node's h row written once (H units), every internal position's operand rows
// (bf16 path) twice - one half per child -, no leaf position's operand row at all.
__global__ void k_check_counts(int n, int H, int bf16, const int* rows, const int* left, const int* counts,
                               DevStatus* st) {
  if (st->status != 0) return;
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n) return;
  bool ok = counts[k] == H;
  if (bf16) {
    // rows[k]: the node whose operand row sits at position k (ready order, or the order by sub-forest)
    const int want = left[chk(st, rows[k], n)] < 0 ? 0 : 2 * H;
    ok = ok && counts[n + k] == want && counts[2 * n + k] == want;
  }
  if (!ok) report(st, TREELSTM_ERR_CHECK);
}
}  // namespace
#endif

int launch_check_clear(treelstm* ctx, int n, void* ws, const WsLayout& lay, cudaStream_t stream) {
#ifdef TREELSTM_CHECKED
  if (n > 0) TL_CUDA(ctx, cudaMemsetAsync(check_counters(ws, lay), 0, sizeof(int) * 3 * (size_t)n, stream));
#else
  (void)ctx; (void)n; (void)ws; (void)lay; (void)stream;
#endif
  return TREELSTM_OK;
}

int launch_check_counts(treelstm* ctx, int n, const int32_t* rows, const int32_t* left, void* ws, const WsLayout& lay,
                        cudaStream_t stream) {
#ifdef TREELSTM_CHECKED
  if (n > 0) {
    DevStatus* st = reinterpret_cast<DevStatus*>(static_cast<char*>(ws) + lay.status);
    k_check_counts<<<(n + 255) / 256, 256, 0, stream>>>(n, ctx->H, ctx->precision == TREELSTM_BF16 ? 1 : 0,
                                                        rows, left, check_counters(ws, lay), st);
    TL_CUDA(ctx, cudaGetLastError());
  }
#else
  (void)ctx; (void)n; (void)rows; (void)left; (void)ws; (void)lay; (void)stream;
#endif
  return TREELSTM_OK;
}

int launch_gather_roots(treelstm* ctx, int max_roots, int32_t* root_ids, float* root_h,
                        float* root_c, int32_t* n_roots, cudaStream_t stream) {
  const auto& L = ctx->last;
  char* base = static_cast<char*>(L.ws);
  const DevStatus* st = reinterpret_cast<const DevStatus*>(base + L.lay.status);
  const int* roots = reinterpret_cast<const int*>(base + L.lay.roots);
  int blocks = max_roots < 1 ? 1 : (max_roots < 1184 ? max_roots : 1184);
  k_gather_roots<<<blocks, 128, 0, stream>>>(max_roots, ctx->H, roots, L.h, L.c, root_ids, root_h,
                                             L.c ? root_c : nullptr, n_roots, st);
  ctx->launches += 1;
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

}  // namespace tl

// ------------------------------------------------------------------------------------------ //
// Scheduling without any allocation: the scratch of the single-CTA scheduler in a fixed array of
// the device image.  Layout: control block | parent | order_tmp | roots, each for
// TREELSTM_STATIC_MAX_NODES nodes.
// ------------------------------------------------------------------------------------------ //
namespace {
constexpr size_t kStaticNodes = TREELSTM_STATIC_MAX_NODES;
constexpr size_t kStaticBytes = sizeof(tl::DevStatus) + 3 * sizeof(int) * kStaticNodes;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

constexpr int kMaxDevices = 64;
unsigned char* g_static_scratch_addr[kMaxDevices] = {};   // device address per device ordinal
}  // namespace

extern "C" int treelstm_schedule_static(int n_nodes, const int32_t* left, const int32_t* right,
                                        const int32_t* token, int vocab, int32_t* level,
                                        int32_t* order, int32_t* level_offset, int32_t* n_levels,
                                        int32_t* status, void* stream) {
  using namespace tl;
  if (n_nodes < 0 || vocab <= 0 || !level_offset || !n_levels || !status) return TREELSTM_ERR_INVALID_ARG;
  if (n_nodes > 0 && (!left || !right || !token || !level || !order)) return TREELSTM_ERR_INVALID_ARG;
  if (n_nodes > TREELSTM_STATIC_MAX_NODES) return TREELSTM_ERR_UNSUPPORTED;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TREELSTM_ERR_NO_DEVICE;
  if (!g_static_scratch_addr[dev]) {
    // In host code the array's name is only a handle for the symbol; the address the kernel can
    // use has to be asked for, once per device, with that device current.
    void* addr = nullptr;
    if (cudaGetSymbolAddress(&addr, g_static_scratch) != cudaSuccess || !addr) return TREELSTM_ERR_CUDA;
    if (cudaFuncSetAttribute(k_schedule_single, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)single_smem_bytes(kSchedSingleMaxNodes, false)) != cudaSuccess)
      return TREELSTM_ERR_CUDA;
    g_static_scratch_addr[dev] = static_cast<unsigned char*>(addr);
  }
  unsigned char* base = g_static_scratch_addr[dev];
  DevStatus* st = reinterpret_cast<DevStatus*>(base);
  int* parent = reinterpret_cast<int*>(base + sizeof(DevStatus));
  int* order_tmp = parent + kStaticNodes;
  int* roots = order_tmp + kStaticNodes;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (n_nodes > 0) {
    // the control block keeps the previous call's status and counts; the kernel's first step is
    // to clear it, everything else in the array is rewritten before it is read
    const bool cache = single_caches_children(n_nodes, false);
    k_schedule_single<<<1, kSingleThreads, single_smem_bytes(n_nodes, false) + (cache ? (size_t)n_nodes * 4 + 16 : 0), s>>>(
        n_nodes, left, right, token, vocab, parent, level, order, order_tmp, level_offset, roots, n_levels, st,
        0, nullptr, nullptr, nullptr, cache ? 1 : 0);
    if (cudaGetLastError() != cudaSuccess) return TREELSTM_ERR_CUDA;
  } else {
    if (cudaMemsetAsync(st, 0, sizeof(DevStatus), s) != cudaSuccess ||
        cudaMemsetAsync(level_offset, 0, sizeof(int32_t), s) != cudaSuccess ||
        cudaMemsetAsync(n_levels, 0, sizeof(int32_t), s) != cudaSuccess)
      return TREELSTM_ERR_CUDA;
  }
  if (cudaMemcpyAsync(status, &st->status, sizeof(int), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
    return TREELSTM_ERR_CUDA;
  return TREELSTM_OK;
}
