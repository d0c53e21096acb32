// The narrow wavefronts at the end of a forest on ONE thread-block cluster, without a trip through
// global memory between a node and its caller (sm_100a: tcgen05.mma, tensor memory, TMA, distributed
// shared memory).
//
// Paper: Section 4.1.1 - a node is ready the moment its inputs are resolved; Section 6.3 - on deep,
// narrow trees only one or two nodes are ready at a time, so what counts is the time from "child
// finished" to "caller finished".  In the grid-wide kernel that chain is: states to global memory,
// grid barrier, operand rows back through TMA, MMAs, cell update - about 9.5 k cycles per wavefront,
// most of it memory round trips.  Here the chain is MMAs, cell update, and a push of the new bf16 h
// straight into the shared memory of the CTAs that need it next.
//
// Layout of the work.  The cluster has cs CTAs; CTA r owns hidden units [r U, (r + 1) U), U = 8 gpc,
// and keeps the packed recurrent weights of those units (40 gpc rows x 2 Hp) in shared memory for the
// whole kernel.  Operands are swapped with respect to the grid-wide kernel: the weight rows are the
// M side of the MMA (tensor-memory lanes = gate rows), the ready nodes the N side (columns, at most
// 64), so a wavefront of any width up to 64 is one chain of MMAs and its accumulator is spread
// over the lanes of three warps per half.  Every CTA needs the operand rows [h_l | h_r] of ALL nodes
// of a wavefront; they live in one of two shared-memory buffers (K-major, 128-byte swizzle, as TMA
// writes them and the MMA reads them).
//
// How a wavefront's operands get there.  (1) A TMA prefetch of its rows from the global operand
// matrix, issued one wavefront ahead: it brings every half whose child finished two or more
// wavefronts ago (and whatever is there for the other halves).  (2) For a child that finishes in
// the wavefront just before, each CTA pushes its U units of the new h into the row of the caller in
// the next buffer of every CTA of the cluster (st.async: the bytes are counted on an mbarrier of the
// receiving CTA, which knows from the delivery slots how many to expect).  The prefetch must have
// landed before a push may overwrite its stale halves: every CTA tells every other one when its
// prefetch is in (P); and the prefetch may only be issued once the global stores of the wavefront
// before the previous one are visible: every CTA tells every other one when its stores have drained
// (G).  Neither signal is on the critical path; the hardware cluster barrier is not used at all.
// Cell states never leave the CTA that owns their units (shared-memory rows per caller position),
// except as a copy to global memory for callers further up.
//
// The five gates of a hidden unit sit in five different tensor-memory lanes (different threads):
// after bias and activation every thread writes its row of gate values to shared memory (node-major),
// and the 256 epilogue threads pick up (node, unit) pairs from there.
//
// All states are also written to global memory as in the other kernels (h, c per node; bf16 h and
// fp32 c into the caller's operand row), so any later consumer - a wavefront further up, the
// backward pass, the caller of the library - finds them where it expects them.
//
// Warp roles (384 threads): warps 0-7 epilogue (warp w reads tensor-memory lane quadrant w mod 4;
// warps 0-3 take the lower half of the node columns, 4-7 the upper half), warp 8 prefetch producer
// and peer signalling, warp 9 MMA issuer and tensor-memory owner, warps 10-11 fetch the row tables
// and child cell states of the next wavefront.
#include "tc_ptx.cuh"

namespace tl {
namespace {

constexpr int kThreads = kTcThreads;
constexpr int kTailRows = 64;             // most nodes per wavefront
constexpr int kEpiThreads = 256;

// ---- PTX: distributed shared memory, cluster-scope mbarrier operations ---------------------------- //
__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory location in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// arrival on an mbarrier of another CTA; release at cluster scope: what this thread wrote before (and
// what it has observed of its own CTA through a CTA barrier) is visible to whoever acquires the phase
__device__ __forceinline__ void mbar_arrive_remote_release(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// arrival on an mbarrier of another CTA that carries no data of this thread with it (a pure "go ahead")
__device__ __forceinline__ void mbar_arrive_remote_relaxed(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// bounded wait on a barrier that other CTAs complete
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* s_abort, long long limit,
                                                  DevStatus* st) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*s_abort) return false;
    if (clock64() - t0 > limit) {
      *s_abort = 1;
      report(st, TREELSTM_ERR_TIMEOUT);
      return false;
    }
  }
}
// 16 bytes into another CTA's shared memory; the bytes are counted on that CTA's mbarrier
__device__ __forceinline__ void st_async16(uint32_t cluster_addr, uint4 v, uint32_t cluster_mbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "r"(cluster_mbar) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr) : "memory");
}

// Shared-memory plan of one CTA (bytes from the 1024-byte aligned base).
struct TailLayout {
  uint32_t wres, xop, cbuf, rows, bars, total;         // xop: 2 buffers, cbuf: 2 buffers, rows: 2 tables
  uint32_t wres_bytes, xop_bytes, cbuf_bytes, gate_bytes;   // gate_bytes: gate values of a wavefront (inside its operand buffer)
};
__host__ __device__ inline TailLayout tail_layout(int Hp, int gpc) {
  TailLayout L;
  const uint32_t kb = 2u * (uint32_t)Hp / kKBlock, U = 8u * (uint32_t)gpc;
  L.wres_bytes = kb * (uint32_t)gpc * kGColsI * 128u;
  L.xop_bytes = kb * (uint32_t)kTailRows * 128u;          // [K block][64 rows][128 bytes]
  L.cbuf_bytes = (uint32_t)kTailRows * 2u * U * 4u;       // [row][side][U] fp32
  uint32_t off = 0;
  L.wres = off; off += (L.wres_bytes + 1023u) & ~1023u;
  L.xop = off; off += 2u * L.xop_bytes;
  L.cbuf = off; off += 2u * L.cbuf_bytes;
  // Once the MMAs of a wavefront have retired its operand buffer is free until the prefetch of the
  // wavefront after next: it then holds the gate values [node][40 gpc] fp32 and, behind them, the new
  // bf16 h of this CTA's units [node][U] (source of the pushes).
  L.gate_bytes = (uint32_t)kTailRows * (uint32_t)gpc * kGColsI * 4u;
  L.rows = off; off += 2u * 3u * (uint32_t)kTailRows * 4u;   // [buffer][node ids | slots | which children are recent]
  L.bars = off; off += 256u;
  L.total = off + 1024u;                                  // alignment slack
  return L;
}

__global__ void __launch_bounds__(kThreads, 1)
k_fwd_tc_tail(const __grid_constant__ TmapSet maps, const __grid_constant__ SfTmapSet sfm, TcParams p) {
  extern __shared__ unsigned char smem_raw[];
  const int gpc = p.groups_per_cta, U = 8 * gpc, Hp = p.Hp, H = p.H;
  const TailLayout L = tail_layout(Hp, gpc);
  const uint32_t raw_addr = smem_u32(smem_raw);
  const uint32_t base = (raw_addr + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_raw + (base - raw_addr);
  const uint32_t wres_addr = base + L.wres;
  float* cbuf = reinterpret_cast<float*>(base_ptr + L.cbuf);
  int* s_rows = reinterpret_cast<int*>(base_ptr + L.rows);      // [buf][0: node ids, 1: slots, 2: recent children][64]
  uint64_t* bars = reinterpret_cast<uint64_t*>(base_ptr + L.bars);
  // bars: 0,1 TL (prefetch landed)  2,3 XF (pushes landed)  4 G  5,6 P  7 TF  8 TE  9 W (weights)  10 drain
  //       11 E1 (meeting point of the epilogue threads)  12, 14 CB (older child cell states of a wavefront fetched)
  const uint32_t bar0 = smem_u32(bars);
  auto TLb = [&](int b) { return bar0 + 8u * b; };
  auto XFb = [&](int b) { return bar0 + 8u * (2 + b); };
  const uint32_t Gb = bar0 + 8u * 4;
  auto Pb = [&](int b) { return bar0 + 8u * (5 + b); };
  const uint32_t TFb = bar0 + 8u * 7, TEb = bar0 + 8u * 8, Wb = bar0 + 8u * 9, drainb = bar0 + 8u * 10;
  const uint32_t E1b = bar0 + 8u * 11;
  auto CBb = [&](int j) { return bar0 + 8u * (j & 1 ? 14 : 12); };   // by wavefront: a phase every other wavefront
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 16);
  volatile int* s_abort = reinterpret_cast<volatile int*>(s_tmem + 1);
  int* s_cnt = const_cast<int*>(s_abort) + 1;                   // [2][2] nodes that push into each buffer, per fetching warp
  __shared__ int s_first[2];

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_levels_all = ld_volatile(&p.st->n_levels);
  if (n_levels_all <= 0) return;
  const int first_level = tail_first_level(p.level_offset, n_levels_all, p.tail_width, p.tail_min_levels, s_first);
  if (first_level >= n_levels_all) return;          // nothing left for the cluster (the same answer in every CTA)
  const int n_lv = n_levels_all - first_level;
  const uint32_t cs = cluster_size(), rank = cluster_rank();
  const int U0 = (int)rank * U;
  const int kb_int = 2 * Hp / kKBlock;
  const int m_rows = gpc * kGColsI;                 // gate rows of this CTA (tensor-memory lanes in use)
#ifdef TREELSTM_TRACE
  long long* const trace = blockIdx.x == 0 ? p.trace : nullptr;
#endif

  if (tid == 0) {
    for (int b = 0; b < 2; ++b) { mbar_init(TLb(b), 1); mbar_init(XFb(b), 1); mbar_init(Pb(b), cs); }
    mbar_init(Gb, cs);
    mbar_init(TFb, 1);
    mbar_init(TEb, kEpiThreads);
    mbar_init(Wb, 1);
    mbar_init(drainb, 1);
    mbar_init(E1b, kEpiThreads);
    mbar_init(CBb(0), 64);
    mbar_init(CBb(1), 64);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) tmem_alloc(smem_u32(s_tmem), 64);  // one accumulator of up to 64 columns
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *s_tmem;
  // every CTA's barriers exist before anyone signals a peer (the only use of the hardware cluster barrier)
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");

  auto loff = [&](int i) { return __ldg(p.level_offset + first_level + i); };   // wavefront i of this kernel
  const int rows0_begin = loff(0);

  // resident weights: K block kb of this CTA's 40 gpc packed rows at wres + kb * m_rows * 128 bytes
  if (warp == 8 && lane == 0) {
    mbar_arrive_expect_tx(Wb, L.wres_bytes);
    tma_load_3d(wres_addr, &sfm.wres, 0, (int)rank * m_rows, 0, Wb);
    // operands of the first wavefront: everything below it is final (written by the grid-wide kernel)
    mbar_arrive_expect_tx(TLb(0), L.xop_bytes);
    tma_load_3d(base + L.xop, &maps.a[1][0], 0, rows0_begin, 0, TLb(0));
    mbar_arrive_expect_tx(XFb(0), 0);               // no pushes into the first buffer
  }
  // nobody pushes into buffer 0 for its first use either: its "peers may push" phase is completed here,
  // so that the k-th use of either buffer waits for phase k of its barriers
  if (warp == 8 && lane < (int)cs) mbar_arrive_remote_release(map_to_cta(Pb(0), (uint32_t)lane));
  // Tables of a wavefront, fetched by warps 10-11 one wavefront ahead: node ids, delivery slots, and
  // per row which of its two children finished one or two wavefronts before it inside this kernel
  // (bit 0 left, bit 1 right) - the cell states of those children are put into the caller's shared-memory
  // row by this CTA's own epilogue, all older ones are read from the global operand rows.
  auto fetch_rows = [&](int i, int b) {             // called by the 64 threads of warps 10-11
    const int t = tid - 320;
    const int begin = loff(i), end = loff(i + 1), nbeg = i + 1 < n_lv ? end : 0, nend = i + 1 < n_lv ? loff(i + 2) : 0;
    int node = -1, slot = -1, fresh = 0;
    if (begin + t < end) {
      node = chk(p.st, p.order[begin + t], p.n);
      slot = chk_slot(p.st, p.slot[node], p.n);
      const int l = chk(p.st, p.left[node], p.n), r = chk(p.st, p.right[node], p.n);
      const int newest = first_level + i - 2 > first_level ? first_level + i - 2 : first_level;
      fresh = (p.level[l] >= newest ? 1 : 0) | (p.level[r] >= newest ? 2 : 0);
    }
    s_rows[(b * 3 + 0) * kTailRows + t] = node;
    s_rows[(b * 3 + 1) * kTailRows + t] = slot;
    s_rows[(b * 3 + 2) * kTailRows + t] = fresh;
    // how many of these nodes deliver into the next wavefront (their caller is one of its rows)
    const bool pushes = slot >= 0 && (slot >> 1) >= nbeg && (slot >> 1) < nend;
    const unsigned m = __ballot_sync(kFullMask, pushes);
    if (lane == 0) s_cnt[b * 2 + (warp - 10)] = __popc(m);
  };
  // Child cell states of wavefront i that are older than two wavefronts: from the global operand rows
  // into cbuf[b].  Only this CTA ever writes its own units of such a row (here or, below the tail, the
  // grid-wide kernel), and what it wrote for children that old was written before the last CTA barrier.
  auto fetch_cells = [&](int i, int b) {
    const int t = tid - 320;
    const int begin = loff(i), rows = loff(i + 1) - begin;
    float* dst = cbuf + (size_t)b * kTailRows * 2 * U;
    const int* fresh = s_rows + (b * 3 + 2) * kTailRows;
    __syncwarp();
    asm volatile("bar.sync 2, 64;" ::: "memory");   // the flags written by both fetching warps are in
    if ((H & 3) == 0) {                             // 16-byte pieces: (row, side) runs of U floats are aligned
      const int c4 = U / 4, total = rows * 2 * c4;
      for (int e0 = 0; e0 < total; e0 += 64 * 8) {
        float4 v[8];
        bool take[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int e = e0 + j * 64 + t;
          v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          take[j] = false;
          if (e < total) {
            const int pair = e / c4, q = e - pair * c4;         // pair = row * 2 + side
            take[j] = !((fresh[pair >> 1] >> (pair & 1)) & 1);
            if (take[j] && U0 + 4 * q < H)
              v[j] = __ldcg(reinterpret_cast<const float4*>(p.cin + (size_t)(2 * begin + pair) * H + U0 + 4 * q));
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int e = e0 + j * 64 + t;
          if (take[j]) reinterpret_cast<float4*>(dst)[e] = v[j];
        }
      }
    } else {
      const int total = rows * 2 * U;
      for (int e0 = 0; e0 < total; e0 += 64 * 8) {
        float v[8];
        bool take[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int e = e0 + j * 64 + t;
          v[j] = 0.f;
          take[j] = false;
          if (e < total) {
            const int pair = e / U, u = e - pair * U;
            take[j] = !((fresh[pair >> 1] >> (pair & 1)) & 1);
            if (take[j] && U0 + u < H) v[j] = __ldcg(p.cin + (size_t)(2 * begin + pair) * H + U0 + u);
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int e = e0 + j * 64 + t;
          if (take[j]) dst[e] = v[j];
        }
      }
    }
  };
  if (warp >= 10) {
    fetch_rows(0, 0);
    fetch_cells(0, 0);
    mbar_arrive(CBb(0));                            // the fetched cell states of wavefront 0 are in
  }

  // what an epilogue thread keeps of its (node, unit) pairs until their copies to global memory are made
  constexpr int kMaxItems = kTailRows * 24 / kEpiThreads;    // pairs per thread at most (U <= 24)
  float keep_h[kMaxItems], keep_c[kMaxItems];
  int keep_node[kMaxItems], keep_slot[kMaxItems];
  unsigned keep_near = 0;                                    // per pair: bit 2 it: caller in the next wavefront; bit 2 it + 1: or the one after
  int kept = 0;                                              // pairs of the previous wavefront (all threads together)
  // Copies to global memory, for callers further up than the shared-memory hand-over reaches and for
  // whoever reads the states later.  The bf16 h in the caller's operand row is what a later prefetch
  // reads (not needed if the caller sits in the next wavefront: it got the push): it goes out right
  // after the pushes, before the CTA's per-wavefront barrier, so that the "copies are out" signal can
  // follow that barrier at once.  The rest (h and c at the node id; c in the caller's row unless the
  // caller is one or two wavefronts up and got it in shared memory) waits until the next wavefront's
  // MMAs run.
  auto copy_operand_rows = [&]() {
#pragma unroll
    for (int it = 0; it < kMaxItems; ++it) {
      const int q = tid + it * kEpiThreads;
      if (q >= kept) break;
      const int unit = U0 + q % U, slot = keep_slot[it];
      if (slot >= 0 && !((keep_near >> (2 * it)) & 1u))
        p.ain[(size_t)slot * Hp + unit] = __float2bfloat16_rn(unit < H ? keep_h[it] : 0.f);
    }
    asm volatile("fence.proxy.async.global;" ::: "memory");    // the operand rows are read through TMA later
  };
  auto copy_states = [&]() {
#pragma unroll
    for (int it = 0; it < kMaxItems; ++it) {
      const int q = tid + it * kEpiThreads;
      if (q >= kept) break;
      const int unit = U0 + q % U;
      if (unit >= H) continue;
      const int node = keep_node[it], slot = keep_slot[it];
      const float hn = keep_h[it], cn = keep_c[it];
      p.h[(size_t)node * H + unit] = hn;
      p.c[(size_t)node * H + unit] = cn;
      count_write(p.chk_counts, node, 1);
      if (slot >= 0) {
        if (!((keep_near >> (2 * it)) & 3u)) p.cin[(size_t)slot * H + unit] = cn;
        count_write(p.chk_counts ? p.chk_counts + p.n : nullptr, slot >> 1, 1);   // handed over, in shared or global memory
        count_write(p.chk_counts ? p.chk_counts + 2 * p.n : nullptr, slot >> 1, 1);
      }
    }
  };

  bool alive = true;
  uint32_t e1_phase = 0;                                        // parity of the epilogue's meeting point
  for (int i = 0; i < n_lv; ++i) {
    const int cur = i & 1, nxt = cur ^ 1;
    const uint32_t use = (uint32_t)(i >> 1) & 1u;                 // parity of this use of buffer `cur`
    const uint32_t use_nxt = (uint32_t)((i + 1) >> 1) & 1u;       // parity of the next use of buffer `nxt`
    const int begin = loff(i), end = loff(i + 1);
    const int rows = end - begin;
    const int n_pad = (rows + 15) & ~15;                          // UMMA N
    const bool more = i + 1 < n_lv;
    const int nbeg = end, nend = more ? loff(i + 2) : end;        // rows of the next wavefront
    const int nend2 = i + 2 < n_lv ? loff(i + 3) : nend;          // and of the one after: [nend, nend2)
    // S0: the tables of this wavefront are in shared memory, the previous wavefront has left this CTA's
    // shared memory.  The MMA warp does not take part: its operands and its accumulator have barriers of
    // their own.  The other warps decide together (an OR over the barrier) whether to go on, so that none
    // of them is left waiting at this barrier by one that saw the flag a moment later.
    if (warp != 9) {
      uint32_t stop_all;
      asm volatile(
          "{\n\t.reg .pred p, q;\n\t"
          "setp.ne.u32 q, %1, 0;\n\t"
          "bar.red.or.pred p, 1, %2, q;\n\t"
          "selp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(stop_all) : "r"((uint32_t)*s_abort), "r"(kThreads - 32) : "memory");
      if (stop_all) break;
    } else if (*s_abort) {
      break;
    }
#ifdef TREELSTM_TRACE
    if (tid == 0) TL_STAMP(trace, first_level + i, 0);
#endif

    if (warp == 8) {
      // ---------------- prefetch of the next wavefront's operand rows, peer signalling ----------------
      if (more) {
        bool ok = true;
        if (lane == 0) {
          // the copies every CTA made of wavefront i - 1 are visible (those of older wavefronts were before)
          ok = mbar_wait_cluster(Gb, (uint32_t)i & 1u, s_abort, p.wait_limit, p.st);
          if (ok) {
            asm volatile("fence.proxy.async;" ::: "memory");   // global rows written, shared buffer last touched, by ordinary stores
            mbar_arrive_expect_tx(XFb(nxt), (uint32_t)(s_cnt[cur * 2] + s_cnt[cur * 2 + 1]) * (uint32_t)(gpc * 16) * cs);
            mbar_arrive_expect_tx(TLb(nxt), L.xop_bytes);
            tma_load_3d(base + L.xop + (uint32_t)nxt * L.xop_bytes, &maps.a[1][0], 0, nbeg, 0, TLb(nxt));
#ifdef TREELSTM_TRACE
            TL_STAMP(trace, first_level + i, 1);
#endif
            ok = mbar_wait(TLb(nxt), use_nxt, s_abort, p.wait_limit, p.st);
#ifdef TREELSTM_TRACE
            TL_STAMP(trace, first_level + i, 7);
#endif
          }
        }
        ok = __shfl_sync(kFullMask, (int)ok, 0) != 0;
        // the prefetch is in (lane 0 has seen its barrier flip): peers may now overwrite the halves their
        // wavefront produces
        if (ok && lane < (int)cs) mbar_arrive_remote_relaxed(map_to_cta(Pb(nxt), (uint32_t)lane));
      }
    } else if (warp == 9) {
      // ---------------- MMA issuer ----------------
      if (lane == 0) {
        if (i == 0 && !mbar_wait(Wb, 0, s_abort, p.wait_limit, p.st)) alive = false;
        if (alive && !mbar_wait(TLb(cur), use, s_abort, p.wait_limit, p.st)) alive = false;
        if (alive && !mbar_wait_cluster(XFb(cur), use, s_abort, p.wait_limit, p.st)) alive = false;
        if (alive && i > 0 && !mbar_wait(TEb, (uint32_t)(i - 1) & 1u, s_abort, p.wait_limit, p.st)) alive = false;
        if (alive) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // pushed pieces are read by the tensor core
          tc_fence_after();
#ifdef TREELSTM_TRACE
          TL_STAMP(trace, first_level + i, 2);
#endif
          const uint32_t idesc = umma_idesc(n_pad);
          const uint32_t x_addr = base + L.xop + (uint32_t)cur * L.xop_bytes;
          for (int kb = 0; kb < kb_int; ++kb) {
            const uint64_t a_desc = umma_desc(wres_addr + (uint32_t)kb * (uint32_t)m_rows * 128u);
            const uint64_t b_desc = umma_desc(x_addr + (uint32_t)kb * (uint32_t)kTailRows * 128u);
#pragma unroll
            for (int k = 0; k < kKBlock / 16; ++k)
              umma_bf16(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, !(kb == 0 && k == 0));
          }
          umma_commit(TFb);
#ifdef TREELSTM_TRACE
          TL_STAMP(trace, first_level + i, 3);
#endif
        }
      }
    } else if (warp >= 10) {
      // ---------------- tables and older child cell states of the next wavefront ----------------
      if (more) {
        fetch_rows(i + 1, nxt);
#ifdef TREELSTM_TRACE
        if (tid == 320) TL_STAMP(trace, first_level + i, 12);
#endif
        fetch_cells(i + 1, nxt);
#ifdef TREELSTM_TRACE
        if (tid == 320) TL_STAMP(trace, first_level + i, 13);
#endif
      }
      mbar_arrive(CBb(i + 1));                      // (two barriers in turn: the epilogue may still have to look at this wavefront's)
    } else {
      // ---------------- epilogue ----------------
      // (a) the operand rows of the previous wavefront went to global memory before S0: every CTA of the
      //     cluster is told (warp 7 has nothing to do with the gate rows); then the rest of that
      //     wavefront's copies, while this wavefront's MMAs run
      if (warp == 7 && lane < (int)cs) mbar_arrive_remote_release(map_to_cta(Gb, (uint32_t)lane));
      if (alive && kept > 0) copy_states();
#ifdef TREELSTM_TRACE
      if (tid == 0) TL_STAMP(trace, first_level + i, 14);
#endif
      // (b) this thread's (node, unit) pairs of the wavefront: where their gates, child cell states and
      //     results live
      const int* s_node = s_rows + (cur * 3 + 0) * kTailRows;
      const int* s_slot = s_rows + (cur * 3 + 1) * kTailRows;
      const int n_items = rows * U;
      int it_g[kMaxItems], it_c[kMaxItems], dep1[kMaxItems], dep2[kMaxItems];
      unsigned near_now = 0;
#pragma unroll
      for (int it = 0; it < kMaxItems; ++it) {
        const int q = tid + it * kEpiThreads;
        it_g[it] = -1; dep1[it] = -1; dep2[it] = -1; it_c[it] = 0;
        if (q < n_items) {
          const int r = q / U, u = q - r * U;
          it_g[it] = r * m_rows + (u >> 3) * kGColsI + (u & 7);
          it_c[it] = r * 2 * U + u;
          const int slot = s_slot[r];
          keep_node[it] = s_node[r];
          keep_slot[it] = slot;
          if (slot >= 0) {
            const int pos = slot >> 1, off = (slot & 1) * U + u;
            if (pos >= nbeg && pos < nend) { dep1[it] = (pos - nbeg) * 2 * U + off; near_now |= 1u << (2 * it); }          // caller in the next wavefront
            else if (pos >= nend && pos < nend2) { dep2[it] = (pos - nend) * 2 * U + off; near_now |= 2u << (2 * it); }    // caller in the one after
          }
        }
      }
      const int e = warp >> 2, quad = warp & 3;
      const int m = quad * 32 + lane;                              // gate row of this thread
      const int half_cols = n_pad >> 1;                            // columns per half: 8, 16, 24 or 32
      const int col0 = e * half_cols;
      const bool active = m < m_rows;
      const float bias = active ? __ldg(p.bp_h + (int)rank * m_rows + m) : 0.f;
      const bool is_tanh = (m % kGColsI) >= 32;                    // rows 32..39 of a group: candidate u
      const float a_in = is_tanh ? 1.f : 0.5f, a_mul = is_tanh ? 1.f : 0.5f, a_add = is_tanh ? 0.f : 0.5f;
      if (!mbar_wait(TFb, (uint32_t)i & 1u, s_abort, p.wait_limit, p.st)) alive = false;
      alive = __all_sync(kFullMask, alive);
      kept = 0;
      if (alive) {
        tc_fence_after();
#ifdef TREELSTM_TRACE
        if (tid == 0) TL_STAMP(trace, first_level + i, 4);
#endif
        // (c) gate values of this row for the nodes of this half -> shared memory, node-major (the operand
        //     buffer of this wavefront is free: its MMAs have retired)
        float* gsm = reinterpret_cast<float*>(base_ptr + L.xop + (size_t)cur * L.xop_bytes);
        __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(base_ptr + L.xop + (size_t)cur * L.xop_bytes + L.gate_bytes);
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)col0;
        uint32_t v[4][8];
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c * 8 < half_cols) tmem_ld8(taddr + (uint32_t)(c * 8), v[c]);   // all loads in flight, one wait
        tmem_ld_wait();
        if (active) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (c * 8 >= half_cols) break;
#pragma unroll
            for (int j = 0; j < 8; ++j) {
              const float z = __uint_as_float(v[c][j]) + bias;
              gsm[(size_t)(col0 + c * 8 + j) * m_rows + m] = fmaf(a_mul, act_tanh(a_in * z), a_add);
            }
          }
        }
        tc_fence_before();
        mbar_arrive(TEb);                                          // the accumulator may be overwritten
        mbar_arrive(E1b);                                          // every gate row is in shared memory
        bool ok = mbar_wait(E1b, e1_phase, s_abort, p.wait_limit, p.st);
        e1_phase ^= 1u;
#ifdef TREELSTM_TRACE
        if (tid == 0) TL_STAMP(trace, first_level + i, 8);
#endif
        ok = mbar_wait(CBb(i), use, s_abort, p.wait_limit, p.st) && ok;   // this wavefront's older cell states are in
#ifdef TREELSTM_TRACE
        if (tid == 0) TL_STAMP(trace, first_level + i, 9);
#endif
        // (d) five gates from shared memory, child cell states, new c and h.  What the next wavefront needs
        //     goes to shared memory at once: bf16 h for the pushes, c into the caller's row.
        const float* ccur = cbuf + (size_t)cur * kTailRows * 2 * U;
        float* cnext = cbuf + (size_t)nxt * kTailRows * 2 * U;
        float* cafter = cbuf + (size_t)cur * kTailRows * 2 * U;    // the buffer of the wavefront after next, once this one has been read
        if (ok) {
#pragma unroll
          for (int it = 0; it < kMaxItems; ++it) {
            if (it_g[it] < 0) break;
            const int q = tid + it * kEpiThreads;
            const float* gr = gsm + it_g[it];
            const float gi = gr[0], gfl = gr[8], gfr = gr[16], go = gr[24], gu = gr[32];
            const float cl = ccur[it_c[it]], cr = ccur[it_c[it] + U];
            const float cn = gi * gu + gfl * cl + gfr * cr;
            const float hn = go * act_tanh(cn);
            const bool real = U0 + (q % U) < H;
            keep_h[it] = hn; keep_c[it] = cn;
            hs[q] = __float2bfloat16_rn(real ? hn : 0.f);
            if (dep1[it] >= 0) cnext[dep1[it]] = real ? cn : 0.f;
            if (p.gates && real) {
              float* gp = p.gates + (size_t)keep_node[it] * 5 * H + U0 + (q % U);
              gp[0] = gi; gp[H] = gfl; gp[2 * H] = gfr; gp[3 * H] = go; gp[4 * H] = gu;
            }
          }
          kept = n_items;
          keep_near = near_now;
        }
#ifdef TREELSTM_TRACE
        if (tid == 0) TL_STAMP(trace, first_level + i, 5);
#endif
        mbar_arrive(E1b);                                          // hs is complete, cbuf[cur] has been read
        ok = mbar_wait(E1b, e1_phase, s_abort, p.wait_limit, p.st) && ok;
        e1_phase ^= 1u;
        if (!ok) alive = false;
#ifdef TREELSTM_TRACE
        if (tid == 0) TL_STAMP(trace, first_level + i, 10);
#endif
        if (ok) {
#pragma unroll
          for (int it = 0; it < kMaxItems; ++it) {
            if (it_g[it] < 0) break;
            if (dep2[it] >= 0) cafter[dep2[it]] = U0 + ((tid + it * kEpiThreads) % U) < H ? keep_c[it] : 0.f;
          }
        }
        if (more) {
          // (e) push: 16-byte pieces (8 units) of the new h into the caller's row of every CTA's next buffer
          ok = mbar_wait_cluster(Pb(nxt), use_nxt, s_abort, p.wait_limit, p.st) && ok;
          ok = __all_sync(kFullMask, ok);
#ifdef TREELSTM_TRACE
          if (tid == 0) TL_STAMP(trace, first_level + i, 11);
#endif
          if (ok) {
            // the cluster size divides the number of epilogue threads: a thread always writes to the same peer
            const uint32_t peer = (uint32_t)tid % cs;
            const uint32_t xnext = map_to_cta(base + L.xop + (uint32_t)nxt * L.xop_bytes, peer);
            const uint32_t xf_peer = map_to_cta(XFb(nxt), peer);
            const int per_pass = kEpiThreads / (int)cs;            // (row, piece) pairs per pass over the threads
            for (int rp = tid / (int)cs; rp < rows * gpc; rp += per_pass) {
              const int r = rp / gpc, ch = rp - r * gpc;
              const int slot = s_slot[r];
              if (slot < 0) continue;
              const int pos = slot >> 1, side = slot & 1;
              if (pos < nbeg || pos >= nend) continue;
              const int rn = pos - nbeg;
              const int k = side * Hp + U0 + ch * 8;                // first of the 8 contraction indices
              const uint32_t off = (uint32_t)(k / kKBlock) * (uint32_t)kTailRows * 128u + (uint32_t)rn * 128u +
                                   ((((uint32_t)(k % kKBlock) >> 3) ^ ((uint32_t)rn & 7u)) << 4);
              const uint4 v = *reinterpret_cast<const uint4*>(hs + r * U + ch * 8);
              st_async16(xnext + off, v, xf_peer);
            }
          } else {
            alive = false;
          }
#ifdef TREELSTM_TRACE
          if (tid == 0) TL_STAMP(trace, first_level + i, 6);
#endif
        }
        if (alive && kept > 0) copy_operand_rows();
      }
    }
  }
  // the last wavefront's copies
  if (warp < 8 && alive && kept > 0 && !*s_abort) copy_states();

  // teardown
  tc_fence_before();
  __syncthreads();
  if (*s_abort) {
    // a wait expired: give what was requested a bounded time to land, the MMAs a bounded time to retire
    if (warp == 8 && lane == 0) { mbar_drain(Wb, 0); }
    if (warp == 9 && lane == 0) { umma_commit(drainb); mbar_drain(drainb, 0); }
    __syncthreads();
  }
  // no CTA may leave while a peer can still write into its shared memory or signal its barriers
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (warp == 9) {
    tc_fence_after();
    tmem_dealloc(tmem_base, 64);
  }
}

}  // namespace

// Shared-memory need of the tail kernel for this context; 0 if it does not fit.
int tail_smem_bytes(const treelstm* ctx) {
  if (!ctx->sf.ok) return 0;
  const TailLayout L = tail_layout(ctx->Hp, ctx->sf.groups_per_cta);
  const uint32_t U = 8u * (uint32_t)ctx->sf.groups_per_cta;
  if (L.gate_bytes + (uint32_t)kTailRows * U * 2u > L.xop_bytes) return 0;
  return L.total <= 232448u - 64u ? (int)L.total : 0;
}

int init_tail_attributes(treelstm* ctx) {
  const int smem = tail_smem_bytes(ctx);
  if (smem <= 0) return TREELSTM_ERR_UNSUPPORTED;
  TL_CUDA(ctx, cudaFuncSetAttribute(k_fwd_tc_tail, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  TL_CUDA(ctx, cudaFuncSetAttribute(k_fwd_tc_tail, cudaFuncAttributeNonPortableClusterSizeAllowed, 1));
  return TREELSTM_OK;
}

// One cluster finishes the narrow wavefronts the grid-wide kernel (launched before on the same stream
// with the same tail parameters) left.
int launch_forward_bf16_tail(treelstm* ctx, int n, const int32_t* left, const int32_t* right, const int32_t* token,
                             float* h, float* c, const int32_t* order, const int32_t* level_offset_dev, int flags,
                             void* ws, const WsLayout& lay, cudaStream_t stream) {
  if (!ctx->have_tmaps || !ctx->sf.ok || !ctx->tail_ok) return TREELSTM_ERR_STATE;
  char* base = static_cast<char*>(ws);
  TcParams p{};
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
  p.h = h; p.c = c;
  p.gates = (flags & TREELSTM_SAVE_FOR_BACKWARD) ? reinterpret_cast<float*>(base + lay.gates) : nullptr;
  p.st = reinterpret_cast<DevStatus*>(base + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  p.level = ctx->last.level;
  p.n_parts = 0;
  p.groups_per_cta = ctx->sf.groups_per_cta;
  p.tail_width = ctx->opt.tail_width;
  p.tail_min_levels = ctx->opt.tail_min_levels;
  p.tail_launched = 1;
  p.trace = nullptr;
#ifdef TREELSTM_TRACE
  p.trace = reinterpret_cast<long long*>(base + lay.trace) + kTraceSlots * kTraceLevels;
  TL_CUDA(ctx, cudaMemsetAsync(p.trace, 0, sizeof(long long) * kTraceSlots * kTraceLevels, stream));
#endif
  int rc = ensure_operand_tmaps(ctx, ws, n, p.xin, p.ain);
  if (rc != TREELSTM_OK) return rc;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = ctx->sf.cluster_size; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(ctx->sf.cluster_size);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = tail_smem_bytes(ctx);
  cfg.stream = stream;
  cfg.attrs = at; cfg.numAttrs = 1;
  TL_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_fwd_tc_tail, ctx->maps, ctx->sf_maps, p));
  ctx->launches += 1;
  return TREELSTM_OK;
}

}  // namespace tl
