// Pieces shared by the tensor-core wavefront kernels: tile constants, the parameter block, PTX
// wrappers (mbarrier, TMA, tcgen05), operand descriptors and the activations of the bf16 path.
#pragma once

#include "common.cuh"

namespace tl {

constexpr int BM = 128;                 // nodes per tile (UMMA M)
constexpr int kMaxStages = 8;
constexpr int kTcThreads = 384;
constexpr int kABytes = BM * 128;       // one K block (64 bf16) of 128 rows
constexpr int kAccCols = 256;           // accumulator stage stride in tensor-memory columns
constexpr int kAcc2Off = 128;           // second partial accumulator inside a stage (thin tiles only)
constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kMaxG = 4;                // unit groups (of 8 hidden units) per tile
constexpr int kGColsI = 40;             // packed rows per unit group, internal nodes (5 gates)
constexpr int kGColsL = 24;             // packed rows per unit group, leaves (gates i, o, u)
constexpr int kLevelCache = 1024;       // wavefront boundaries kept in shared memory

struct TcParams {
  int n, H, Hp, Ep, sched_ctas, vocab;
  int* chk_counts;               // checked build: write counters [h per node | Ain per position | Cin per position]
  const int *left, *right, *token, *order, *roots, *level_offset;
  int* slot;
  const __nv_bfloat16* emb_bf;
  const __nv_bfloat16 *wp_h = nullptr, *wp_x = nullptr;   // packed weights (grid-wide kernel: warmed into L2 at its start)
  __nv_bfloat16 *xin, *ain;
  float* cin;
  const float *bp_h, *bp_x;
  float *h, *c, *gates;
  DevStatus* st;
  long long wait_limit;
  // sub-forest (cluster) kernel only
  const int *level, *part_offset;
  int* part_level_spill;
  int n_parts, groups_per_cta;   // n_parts == 0: the cluster kernel runs as the tail of the grid-wide kernel
  // hand-over from the grid-wide kernel to one cluster (persistent mode): see tail_first_level
  int tail_width, tail_min_levels;
  int tail_launched;             // the cluster kernel follows on the stream (else the decision is only recorded)
  // grid-wide kernel started under the scheduler: the leaf wavefront is ranked and evaluated before
  // the schedule is read.  pre_counts [grid]: leaves per CTA's share of the node ids; pre_order [n]: the
  // leaves in ascending node id
  int leaves_first = 0;
  int* pre_counts = nullptr;
  int* pre_order = nullptr;
  long long* trace;              // cycle stamps (trace builds), else nullptr
};

// Where the grid-wide kernel stops and one cluster takes over (persistent mode): the first wavefront
// - never the leaves - from which on every wavefront has at most tail_width nodes, if handing those
// over pays.  With tail_min_levels > 0 it pays when at least that many wavefronts remain.  With
// tail_min_levels == 0 a cost model fitted to cycle traces and step times decides: a wavefront of w
// nodes takes the grid-wide kernel about 9.5 k cycles whatever w, the cluster about 5.5 k + 100 w (it
// passes states through shared memory, at a price per node: every CTA of the cluster gets a copy), and
// the hand-over itself - a launch, the cluster's set-up and its first wavefront waiting for the
// weights - about 30 k; the tail goes to the cluster if the wavefronts it takes save more than that.  Returns n_levels if there is no such tail or tail_width
// is 0.  Both kernels call this with the same arguments and take the same decision.  Cooperative over
// the CTA: every thread calls it; s_tmp is two shared ints.
constexpr int kTailGainBase = 4000, kTailGainPerRow = 100, kTailHandOver = 30000;
__device__ __forceinline__ int tail_first_level(const int* level_offset, int n_levels, int tail_width,
                                                int tail_min_levels, int* s_tmp) {
  if (threadIdx.x == 0) { s_tmp[0] = 1; s_tmp[1] = 0; }   // the leaf wavefront always stays with the grid-wide kernel
  __syncthreads();
  int wide_end = 0;                        // 1 + the last wavefront wider than tail_width
  for (int l = threadIdx.x; l < n_levels; l += blockDim.x)
    if (level_offset[l + 1] - level_offset[l] > tail_width) wide_end = l + 1;
  if (wide_end > 1) atomicMax(&s_tmp[0], wide_end);
  __syncthreads();
  const int first = s_tmp[0];
  if (tail_width > 0 && tail_min_levels <= 0) {
    int gain = 0;                          // cycles the cluster saves on the wavefronts from `first` on
    for (int l = first + threadIdx.x; l < n_levels; l += blockDim.x)
      gain += kTailGainBase - kTailGainPerRow * (level_offset[l + 1] - level_offset[l]);
    if (gain != 0) atomicAdd(&s_tmp[1], gain);
  }
  __syncthreads();
  const int gain_all = s_tmp[1];
  __syncthreads();                         // s_tmp may be reused by the caller
  if (tail_width <= 0 || first >= n_levels) return n_levels;
  if (tail_min_levels > 0) return n_levels - first >= tail_min_levels ? first : n_levels;
  return gain_all > kTailHandOver ? first : n_levels;
}

// ---- PTX wrappers ---------------------------------------------------------------------------- //
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok;
}
// Bounded wait: gives up when the cycle budget is spent or another thread of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* s_abort,
                                          long long limit, DevStatus* st) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  for (;;) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*s_abort) return false;
    if (clock64() - t0 > limit) {
      *s_abort = 1;
      report(st, TREELSTM_ERR_TIMEOUT);
      return false;
    }
  }
}
// Teardown after a failed wait: give a barrier whose phase may still complete (bytes of a bulk copy
// in flight, tensor-core work not yet retired) a bounded time to do so, whatever the abort flag says.
constexpr long long kDrainCycles = 400000;   // about 0.2 ms
__device__ __forceinline__ bool mbar_drain(uint32_t bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kDrainCycles) return false;
  }
  return true;
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
// One request for a box of {64 elements, rows, K blocks}: a request costs the TMA unit of an SM
// about 180 cycles whatever its size and requests are served one after the other, so a tile's
// operands are fetched with as few requests as possible.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar) : "memory");
}
// Ask for the 128-byte lines of [ptr, ptr + bytes) to be brought into L2, spread over n_threads threads.
__device__ __forceinline__ void warm_l2(const void* ptr, size_t bytes, int thread, int n_threads) {
  const char* b = static_cast<const char*>(ptr);
  for (size_t off = (size_t)thread * 128; off < bytes; off += (size_t)n_threads * 128)
    asm volatile("prefetch.global.L2 [%0];" ::"l"(b + off));
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t dst_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(dst_smem), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld4(uint32_t taddr, uint32_t* v) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile stored as rows of 128 bytes with the
// 128-byte swizzle (8-row groups of 1024 bytes): start address, stride between 8-row groups,
// descriptor version 1, swizzle mode 2.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
  d |= (uint64_t)1 << 16;                 // leading byte offset (unused for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // version
  d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
  return d;
}
// Instruction descriptor: D fp32, A and B bf16, both K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// Activations of the bf16 path.  tanh.approx has an absolute error of about 5e-4, far inside the
// 3e-2 budget of this path (the operands are already rounded to 8 mantissa bits).
__device__ __forceinline__ float act_tanh(float x) {
  float y;
  asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float act_sigmoid(float x) { return fmaf(0.5f, act_tanh(0.5f * x), 0.5f); }

__device__ __forceinline__ void st_row4(float* p, bool vec, int count, const float* v) {
  if (vec && count == 4) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (j < count) p[j] = v[j];
  }
}

// Xin[row] = emb_bf[token of the leaf at ready position row] for rows [row_begin, row_end), spread over
// n_warps warps.  A warp takes four rows at a time: their order and token entries are fetched side by
// side, then every lane copies 16-byte pieces of the four embedding rows with all its loads in
// flight before the first store - the copy is bound by memory latency, not by bandwidth.
__device__ __forceinline__ void gather_leaf_rows(const TcParams& p, int row_begin, int row_end, int gwarp, int n_warps,
                                                 int lane) {
  const int cpr = p.Ep / 8;                              // 16-byte chunks per row
  for (int base = row_begin + gwarp; base < row_end; base += 4 * n_warps) {
    const int my_row = base + (lane & 3) * n_warps;
    const int my_tok = my_row < row_end ? chk(p.st, p.token[chk(p.st, p.order[my_row], p.n)], p.vocab) : 0;
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
          if (base + k * n_warps < row_end && cc < cpr)
            v[k][h] = __ldg(reinterpret_cast<const uint4*>(p.emb_bf + (size_t)tok[k] * p.Ep) + cc);
        }
#pragma unroll
      for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int cc = c0 + h * 32 + lane;
          if (base + k * n_warps < row_end && cc < cpr)
            reinterpret_cast<uint4*>(p.xin + (size_t)(base + k * n_warps) * p.Ep)[cc] = v[k][h];
        }
    }
  }
}

// Tiled tensor map over a row-major bf16 matrix [rows][inner] seen as {64, rows, inner / 64}: boxes of
// 64 elements x box_rows rows x box_kb K blocks with the 128-byte swizzle (gemm_tc.cu).
int make_tmap(treelstm* ctx, CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint32_t box_rows,
              uint32_t box_kb);

}  // namespace tl
