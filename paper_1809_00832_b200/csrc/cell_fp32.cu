// fp32 wavefront evaluation: for one wavefront (all nodes of one level), gather the operand rows
// through the child arrays / leaf tokens, contract them with W on the FP32 FMA pipes, and apply
// the cell update in the same kernel (no gate matrix is ever written out unless the caller
// wants it kept for backward).
//
// Paper: Figure 2 (Section 3.1) - leaf: LSTM(embed(word)); internal: LSTM(left_state,
// right_state); Section 2.2 - the two child calls are independent, so all nodes whose children
// are done can run together.
#include "common.cuh"

namespace tl {
namespace {

constexpr int TM = 64;       // rows (nodes) per tile on wide wavefronts
constexpr int TMS = 16;      // rows per tile where TM-row tiles would leave most SMs idle
constexpr int TU = 16;       // hidden units per tile (x 5 gates = 80 columns)
constexpr int KC = 32;       // contraction chunk
constexpr int kThreads = 256;
constexpr int kWLoads = KC * 5 * TU / kThreads;    // 10 weight elements per thread and chunk

struct FwdParams {
  int n, H, E, n_sms, vocab;
  int* chk_counts;   // checked build: writes of h per node
  const int *left, *right, *token, *order, *level_offset;
  const float *emb, *W, *b;
  float *h, *c, *gates;
  DevStatus* st;
  long long wait_limit;
  int w_stationary, a_row, w_row;   // persistent kernel: W_h slice resident in shared memory; row strides (floats)
  int early_start = 0;              // persistent kernel: launched under the scheduler, waits for it on the device
  long long* trace = nullptr;       // cycle stamps of the persistent kernel (trace builds), else nullptr
};

__device__ __forceinline__ float sigmoidf_acc(float x) { return 1.0f / (1.0f + expf(-x)); }

constexpr int kChunkRow = KC + 4;   // floats per shared-memory row of a chunk: 16-byte reads along the contraction,
                                    // consecutive rows 4 banks apart (eight rows cover all banks)
struct TileSmem {
  __align__(16) float A[2][TM][kChunkRow];
  __align__(16) float W[2][5 * TU][kChunkRow];   // transposed: one row per gate column
  int node[TM], l[TM], r[TM];
};

// Rows per tile of a wavefront of `rows` nodes: a level-uniform choice.
// (16-row tiles as long as they take at most two rounds over the SMs: a 64-row tile re-uses every
// weight it reads four times, but costs about twice a 16-row one.)
__host__ __device__ inline int rows_per_tile(int rows, int tiles_u, int n_sms) {
  return ((rows + TMS - 1) / TMS) * tiles_u > 2 * n_sms ? TM : TMS;
}

// One tile: rows [row0, row0 + TM) of the ready order (clipped to row_end), hidden units
// [u0, u0 + TU).  `leaf` selects x = emb[token] with W rows [0, E) and gates i, o, u only.
// The next K chunk is fetched into registers while the current one is multiplied out of shared
// memory (two buffers, one CTA barrier per chunk).
template <int TM>
__device__ void fp32_tile(const FwdParams& p, int row0, int row_end, int u0, bool leaf,
                          TileSmem& s, long long* trace = nullptr, int lvl = 0) {
  (void)trace; (void)lvl;
  constexpr int RPT = TM / (kThreads / TU);          // rows per thread: 4 or 1
  constexpr int kALoads = TM * KC / kThreads;        // operand elements per thread and chunk: 8 or 2
  const int tid = threadIdx.x, tx = tid % TU, ty = tid / TU;
  const int H = p.H, E = p.E, K = leaf ? E : 2 * H;
  const float* Wk = p.W + (size_t)(leaf ? 0 : E) * 5 * H;
  __syncthreads();  // previous tile's readers of s are done
  for (int i = tid; i < TM; i += kThreads) {
    const int row = row0 + i;
    int node = -1, l = 0, r = 0;
    if (row < row_end) {
      node = chk(p.st, p.order[row], p.n);
      l = leaf ? chk(p.st, p.token[node], p.vocab) : chk(p.st, p.left[node], p.n);
      r = leaf ? 0 : chk(p.st, p.right[node], p.n);
    }
    s.node[i] = node; s.l[i] = l; s.r[i] = r;
  }
  __syncthreads();
  float acc[RPT][5];
#pragma unroll
  for (int i = 0; i < RPT; ++i)
#pragma unroll
    for (int g = 0; g < 5; ++g) acc[i][g] = 0.f;

  float ra[kALoads], rw[kWLoads];
  // All loads of a chunk without a branch (indices clamped onto valid elements, values discarded afterwards),
  // so that they are in flight together: a load behind a branch waits for the one before it.
  auto fetch = [&](int k0) {
    if (leaf) {
#pragma unroll
      for (int j = 0; j < kALoads; ++j) {
        const int e = tid + j * kThreads, i = e / KC, k = min(k0 + e % KC, K - 1);
        ra[j] = __ldg(p.emb + (size_t)s.l[i] * E + k);
      }
    } else {
#pragma unroll
      for (int j = 0; j < kALoads; ++j) {
        const int e = tid + j * kThreads, i = e / KC, k = min(k0 + e % KC, K - 1);
        ra[j] = __ldcg(p.h + (size_t)(k < H ? s.l[i] : s.r[i]) * H + (k < H ? k : k - H));
      }
    }
#pragma unroll
    for (int j = 0; j < kWLoads; ++j) {
      const int e = tid + j * kThreads, kk = e / (5 * TU), g = (e % (5 * TU)) / TU, uu = e % TU;
      rw[j] = __ldg(Wk + (size_t)min(k0 + kk, K - 1) * 5 * H + g * H + min(u0 + uu, H - 1));
    }
  };
  // (what the clamped loads brought for elements outside the tile is replaced by zeros here, not in fetch: a
  // use of the loaded values right behind the loads would make the multiply-adds of the current chunk wait)
  auto stash = [&](int buf, int k0) {
#pragma unroll
    for (int j = 0; j < kALoads; ++j) {
      const int e = tid + j * kThreads, i = e / KC, k = k0 + e % KC;
      s.A[buf][i][e % KC] = (s.node[i] < 0 || k >= K) ? 0.f : ra[j];
    }
#pragma unroll
    for (int j = 0; j < kWLoads; ++j) {
      const int e = tid + j * kThreads, kk = e / (5 * TU), g = (e % (5 * TU)) / TU, uu = e % TU;
      s.W[buf][e % (5 * TU)][kk] = (k0 + kk >= K || u0 + uu >= H || (leaf && (g == 1 || g == 2))) ? 0.f : rw[j];
    }
  };
  // the bias is asked for now and arrives while the contraction runs
  const int u = u0 + tx;
  float bias[5];
#pragma unroll
  for (int g = 0; g < 5; ++g) bias[g] = __ldg(p.b + g * H + min(u, H - 1));
  TL_STAMP(trace, lvl, 3);   // row ids resolved
  fetch(0);
  stash(0, 0);
  __syncthreads();
  TL_STAMP(trace, lvl, 4);   // first chunk in shared memory
  const int chunks = (K + KC - 1) / KC;
  for (int cidx = 0; cidx < chunks; ++cidx) {
    const int buf = cidx & 1;
    if (cidx + 1 < chunks) fetch((cidx + 1) * KC);
#pragma unroll
    for (int kk = 0; kk < KC; kk += 4) {
      float4 a[RPT], w[5];
#pragma unroll
      for (int i = 0; i < RPT; ++i) a[i] = *reinterpret_cast<const float4*>(&s.A[buf][ty * RPT + i][kk]);
#pragma unroll
      for (int g = 0; g < 5; ++g) w[g] = *reinterpret_cast<const float4*>(&s.W[buf][g * TU + tx][kk]);
#pragma unroll
      for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int g = 0; g < 5; ++g) {
          acc[i][g] = fmaf(a[i].x, w[g].x, acc[i][g]);
          acc[i][g] = fmaf(a[i].y, w[g].y, acc[i][g]);
          acc[i][g] = fmaf(a[i].z, w[g].z, acc[i][g]);
          acc[i][g] = fmaf(a[i].w, w[g].w, acc[i][g]);
        }
    }
    if (cidx + 1 < chunks) stash(buf ^ 1, (cidx + 1) * KC);
    __syncthreads();
  }

  TL_STAMP(trace, lvl, 5);   // contraction done
  if (u >= H) return;
#pragma unroll
  for (int i = 0; i < RPT; ++i) {
    const int ii = ty * RPT + i;
    const int node = s.node[ii];
    if (node < 0) continue;
    const float gi = sigmoidf_acc(acc[i][0] + bias[0]);
    const float go = sigmoidf_acc(acc[i][3] + bias[3]);
    const float gu = tanhf(acc[i][4] + bias[4]);
    float gfl = 0.f, gfr = 0.f, cn = gi * gu;
    if (!leaf) {
      gfl = sigmoidf_acc(acc[i][1] + bias[1]);
      gfr = sigmoidf_acc(acc[i][2] + bias[2]);
      cn += gfl * __ldcg(p.c + (size_t)s.l[ii] * H + u) + gfr * __ldcg(p.c + (size_t)s.r[ii] * H + u);
    }
    p.c[(size_t)node * H + u] = cn;
    p.h[(size_t)node * H + u] = go * tanhf(cn);
    count_write(p.chk_counts, node, 1);
    if (p.gates) {
      float* g = p.gates + (size_t)node * 5 * H + u;
      g[0] = gi; g[H] = gfl; g[2 * H] = gfr; g[3 * H] = go; g[4 * H] = gu;
    }
  }
}

// Internal-node tile of the persistent kernel when the recurrent weights of the CTA's 16 hidden
// units stay in shared memory for the whole kernel (Ws[5 * TU][w_row], one row per gate column, the
// contraction index contiguous): only the operand rows [h_l | h_r] of the tile are fetched, all
// loads of a thread in flight together, and the contraction runs out of shared memory in float4
// steps, every thread on 4 rows x 5 gates of one hidden unit.  A 16-row tile has only 4 such row
// groups, so its 16 thread groups also split the contraction in four; the partial sums meet in
// shared memory (red[4][TMS][5 * TU]).  Same cell update as fp32_tile.
template <int TM>
__device__ void fp32_tile_stationary(const FwdParams& p, int row0, int row_end, int u0, float* As,
                                     const float* Ws, float* red, int* s_node, int* s_l, int* s_r,
                                     bool ids_ready = false) {
  constexpr bool kSplit = TM == TMS;
  constexpr int RPT = 4, NQ = kSplit ? 4 : 1;
  const int tid = threadIdx.x, tx = tid % TU, ty = tid / TU;
  const int rg = kSplit ? (ty & 3) : ty, kq = kSplit ? (ty >> 2) : 0;
  const int H = p.H, K = 2 * H, K4 = (K + 3) & ~3, a_row = p.a_row, w_row = p.w_row;
  __syncthreads();  // previous tile's readers of As, red and the index arrays are done
  for (int i = tid; i < TM && !ids_ready; i += kThreads) {   // ids_ready: fetched while the grid barrier was pending
    const int row = row0 + i;
    int node = -1, l = 0, r = 0;
    if (row < row_end) {
      node = chk(p.st, p.order[row], p.n);
      l = chk(p.st, p.left[node], p.n);
      r = chk(p.st, p.right[node], p.n);
    }
    s_node[i] = node; s_l[i] = l; s_r[i] = r;
  }
  __syncthreads();
  if ((H & 1) == 0) {
    const int hp = H / 2, pairs = K4 / 2;            // float2 pieces per child row / per operand row
    const int total = TM * pairs;
    for (int base = 0; base < total; base += 8 * kThreads) {
      float2 v[8];
      int dst[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int e = base + j * kThreads + tid;
        v[j] = make_float2(0.f, 0.f);
        dst[j] = -1;
        if (e < total) {
          const int i = e / pairs, q = e - i * pairs;
          dst[j] = i * a_row + 2 * q;
          if (s_node[i] >= 0 && q < 2 * hp) {
            const float* src = q < hp ? p.h + (size_t)s_l[i] * H + 2 * q : p.h + (size_t)s_r[i] * H + 2 * (q - hp);
            v[j] = __ldcg(reinterpret_cast<const float2*>(src));
          }
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (dst[j] >= 0) *reinterpret_cast<float2*>(As + dst[j]) = v[j];
    }
  } else {
    const int total = TM * K4;
    for (int base = 0; base < total; base += 8 * kThreads) {
      float v[8];
      int dst[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int e = base + j * kThreads + tid;
        v[j] = 0.f;
        dst[j] = -1;
        if (e < total) {
          const int i = e / K4, k = e - i * K4;
          dst[j] = i * a_row + k;
          if (s_node[i] >= 0 && k < K)
            v[j] = k < H ? __ldcg(p.h + (size_t)s_l[i] * H + k) : __ldcg(p.h + (size_t)s_r[i] * H + (k - H));
        }
      }
#pragma unroll
      for (int j = 0; j < 8; ++j)
        if (dst[j] >= 0) As[dst[j]] = v[j];
    }
  }
  __syncthreads();
  float acc[RPT][5];
#pragma unroll
  for (int i = 0; i < RPT; ++i)
#pragma unroll
    for (int g = 0; g < 5; ++g) acc[i][g] = 0.f;
  // what the cell update needs beside the contraction is asked for now and arrives while it runs: the bias
  // and the children's cell states of the rows this thread will finish (row ty of a split tile, else its four)
  const int u = u0 + tx;
  float bias[5] = {};
  constexpr int kFin = kSplit ? 1 : RPT;
  float c_left[kFin], c_right[kFin];
  if (u < H) {
#pragma unroll
    for (int g = 0; g < 5; ++g) bias[g] = __ldg(p.b + g * H + u);
  }
#pragma unroll
  for (int i = 0; i < kFin; ++i) {
    const int ii = kSplit ? ty : rg * RPT + i;
    const bool valid = u < H && s_node[ii] >= 0;
    c_left[i] = valid ? __ldcg(p.c + (size_t)s_l[ii] * H + u) : 0.f;
    c_right[i] = valid ? __ldcg(p.c + (size_t)s_r[ii] * H + u) : 0.f;
  }
  const int steps = K4 / 4, per = (steps + NQ - 1) / NQ;
  const int k_lo = kq * per * 4, k_hi = min(K4, k_lo + per * 4);
  for (int k = k_lo; k < k_hi; k += 4) {
    float4 a[RPT], w[5];
#pragma unroll
    for (int i = 0; i < RPT; ++i) a[i] = *reinterpret_cast<const float4*>(As + (rg * RPT + i) * a_row + k);
#pragma unroll
    for (int g = 0; g < 5; ++g) w[g] = *reinterpret_cast<const float4*>(Ws + (g * TU + tx) * w_row + k);
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
      for (int g = 0; g < 5; ++g) {
        acc[i][g] = fmaf(a[i].x, w[g].x, acc[i][g]);
        acc[i][g] = fmaf(a[i].y, w[g].y, acc[i][g]);
        acc[i][g] = fmaf(a[i].z, w[g].z, acc[i][g]);
        acc[i][g] = fmaf(a[i].w, w[g].w, acc[i][g]);
      }
  }
  auto finish = [&](int ii, const float* z, float cl, float cr) {   // cell update of tile row ii, hidden unit u
    const int node = s_node[ii];
    if (node < 0 || u >= H) return;
    const float gi = sigmoidf_acc(z[0] + bias[0]);
    const float gfl = sigmoidf_acc(z[1] + bias[1]);
    const float gfr = sigmoidf_acc(z[2] + bias[2]);
    const float go = sigmoidf_acc(z[3] + bias[3]);
    const float gu = tanhf(z[4] + bias[4]);
    const float cn = gi * gu + gfl * cl + gfr * cr;
    p.c[(size_t)node * H + u] = cn;
    p.h[(size_t)node * H + u] = go * tanhf(cn);
    count_write(p.chk_counts, node, 1);
    if (p.gates) {
      float* g = p.gates + (size_t)node * 5 * H + u;
      g[0] = gi; g[H] = gfl; g[2 * H] = gfr; g[3 * H] = go; g[4 * H] = gu;
    }
  };
  if (kSplit) {
    // partial sums of the four quarters of the contraction meet here; thread (tx, ty) then finishes row ty
#pragma unroll
    for (int i = 0; i < RPT; ++i)
#pragma unroll
      for (int g = 0; g < 5; ++g) red[(kq * TMS + rg * RPT + i) * (5 * TU) + g * TU + tx] = acc[i][g];
    __syncthreads();
    float z[5];
#pragma unroll
    for (int g = 0; g < 5; ++g) {
      float sum = 0.f;
#pragma unroll
      for (int q = 0; q < NQ; ++q) sum += red[(q * TMS + ty) * (5 * TU) + g * TU + tx];
      z[g] = sum;
    }
    finish(ty, z, c_left[0], c_right[0]);
  } else {
#pragma unroll
    for (int i = 0; i < RPT; ++i) finish(rg * RPT + i, acc[i], c_left[i], c_right[i]);
  }
}

__global__ void __launch_bounds__(kThreads)
k_fwd_fp32_level(FwdParams p, int row_begin, int row_end, int leaf) {
  __shared__ TileSmem s;
  const int tiles_u = (p.H + TU - 1) / TU;
  const int tm = blockIdx.x / tiles_u, tu = blockIdx.x % tiles_u;
  const int tmr = rows_per_tile(row_end - row_begin, tiles_u, p.n_sms);
  if (tmr == TM) fp32_tile<TM>(p, row_begin + tm * TM, row_end, tu * TU, leaf != 0, s);
  else fp32_tile<TMS>(p, row_begin + tm * TMS, row_end, tu * TU, leaf != 0, s);
}

// All wavefronts in one cooperative launch; a bounded grid barrier separates the levels.
// Dynamic shared memory: [operand rows of a tile, at least a TileSmem][resident W_h slice][partial sums][row ids].
__global__ void __launch_bounds__(kThreads)
k_fwd_fp32_persistent(FwdParams p) {
  extern __shared__ float4 dyn_smem[];
  __shared__ int s_flag;
  TileSmem& s = *reinterpret_cast<TileSmem*>(dyn_smem);
  float* As = reinterpret_cast<float*>(dyn_smem);
  size_t a_floats = (size_t)TM * p.a_row;
  if (a_floats * 4 < sizeof(TileSmem)) a_floats = (sizeof(TileSmem) + 3) / 4;
  a_floats = (a_floats + 3) & ~(size_t)3;
  float* Ws = As + a_floats;
  float* red = Ws + (p.w_stationary ? (size_t)5 * TU * p.w_row : 0);          // [4][TMS][5 * TU] partial sums
  int* s_node = reinterpret_cast<int*>(red + (p.w_stationary ? 4 * TMS * 5 * TU : 0));
  int* s_l = s_node + TM;
  int* s_r = s_l + TM;
  const int tiles_u = (p.H + TU - 1) / TU;
  const int H = p.H;
#ifdef TREELSTM_TRACE
  // first CTA, first thread: row l = wavefront l (slot 0 start, 1 own tiles done, 2 barrier passed); last row: phases
  long long* const trace = blockIdx.x == 0 && threadIdx.x == 0 ? p.trace : nullptr;
#endif
  TL_STAMP(trace, kTraceLevels - 1, 0);
  // Launched as a programmatic dependent of the ready-set construction (p.early_start), the kernel
  // gets here while that one still runs: the weight slice needs nothing from it and is fetched first.
  int n_levels = 0;
  if (!p.early_start) {
    if (ld_volatile(&p.st->status) != 0) return;
    n_levels = p.st->n_levels;
  }
  if (p.w_stationary && (p.early_start || n_levels > 1)) {
    // The grid is a multiple of tiles_u, so tile t of any level, t = blockIdx.x + i * gridDim.x, has
    // the same hidden-unit slice: its rows of W_h are fetched once, transposed to [column][k].
    const int u0 = (blockIdx.x % tiles_u) * TU, K = 2 * H, w_row = p.w_row;
    const float* Wk = p.W + (size_t)p.E * 5 * H;
    for (int e = threadIdx.x; e < 5 * TU * w_row; e += kThreads) {
      const int k = e / (5 * TU), col = e - k * 5 * TU, g = col / TU, uu = col - g * TU;
      float v = 0.f;
      if (k < K && u0 + uu < H) v = __ldg(Wk + (size_t)k * 5 * H + g * H + u0 + uu);
      Ws[col * w_row + k] = v;
    }
  }
  {
    // The leaf wavefront streams W_x and the leaves' embedding rows chunk by chunk, one dependent fetch per
    // chunk: asked into L2 now (which nodes are leaves and their tokens are the caller's arrays, readable
    // before the schedule exists; tokens are clamped, nothing has been validated yet), those fetches find
    // them there instead of in DRAM.
    const size_t gthread = (size_t)blockIdx.x * kThreads + threadIdx.x, gthreads = (size_t)gridDim.x * kThreads;
    const char* wx = reinterpret_cast<const char*>(p.W);
    const size_t wx_bytes = sizeof(float) * (size_t)p.E * 5 * H;
    for (size_t off = gthread * 128; off < wx_bytes; off += gthreads * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(wx + off));
    const int lane = threadIdx.x & 31;
    const int row_lines = (int)((sizeof(float) * (size_t)p.E + 127) / 128) + 1;   // + 1: rows do not start on a line
    for (int node = (int)(gthread >> 5); node < p.n; node += (int)(gthreads >> 5)) {
      if (p.left[node] >= 0) continue;
      const int tok = min(max(p.token[node], 0), p.vocab - 1);
      const char* row = reinterpret_cast<const char*>(p.emb + (size_t)tok * p.E);
      for (int l = lane; l < row_lines; l += 32) {
        const char* q = row + (size_t)l * 128;
        if (q < row + sizeof(float) * (size_t)p.E) asm volatile("prefetch.global.L2 [%0];" ::"l"(q));
      }
    }
  }
  TL_STAMP(trace, kTraceLevels - 1, 1);   // weight slice requested (own part stored)
  if (p.early_start) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (ld_volatile(&p.st->status) != 0) return;
    n_levels = p.st->n_levels;
  }
  TL_STAMP(trace, kTraceLevels - 1, 2);   // schedule there
  // the first wavefront boundaries in shared memory: no dependent global load after every barrier
  constexpr int kOffCache = 256;
  __shared__ int s_off[kOffCache];
  for (int i = threadIdx.x; i < kOffCache && i <= n_levels; i += kThreads) s_off[i] = p.level_offset[i];
  __syncthreads();
  auto level_begin = [&](int l) { return l < kOffCache ? s_off[l] : p.level_offset[l]; };
  bool ids_ahead = false;   // uniform: the row ids of this CTA's first tile of the wavefront are in shared memory
  for (int lvl = 0; lvl < n_levels; ++lvl) {
    const int begin = level_begin(lvl), end = level_begin(lvl + 1);
    const int tmr = rows_per_tile(end - begin, tiles_u, p.n_sms);
    const int tiles = ((end - begin + tmr - 1) / tmr) * tiles_u;
    TL_STAMP(trace, lvl, 0);
    for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
      const int tm = t / tiles_u, u0 = (t - tm * tiles_u) * TU;
      if (lvl > 0 && p.w_stationary) {
        const bool ready = ids_ahead && t == (int)blockIdx.x;
        if (tmr == TM) fp32_tile_stationary<TM>(p, begin + tm * TM, end, u0, As, Ws, red, s_node, s_l, s_r, ready);
        else fp32_tile_stationary<TMS>(p, begin + tm * TMS, end, u0, As, Ws, red, s_node, s_l, s_r, ready);
      } else {
#ifdef TREELSTM_TRACE
        if (tmr == TM) fp32_tile<TM>(p, begin + tm * TM, end, u0, lvl == 0, s, trace, lvl);
        else fp32_tile<TMS>(p, begin + tm * TMS, end, u0, lvl == 0, s, trace, lvl);
#else
        if (tmr == TM) fp32_tile<TM>(p, begin + tm * TM, end, u0, lvl == 0, s);
        else fp32_tile<TMS>(p, begin + tm * TMS, end, u0, lvl == 0, s);
#endif
      }
    }
    TL_STAMP(trace, lvl, 1);
    if (lvl + 1 < n_levels) {
      // Which rows the next wavefront holds and who their children are is the scheduler's output and
      // does not depend on the wavefront just finished: threads outside the polling warp fetch the
      // ids of this CTA's first tile of the next wavefront while the barrier is pending (three
      // dependent loads off the path that follows the barrier).
      const bool passed = grid_barrier_with(
          p.st, (unsigned)(lvl + 1) * gridDim.x, p.wait_limit, &s_flag, true, nullptr, nullptr, [&]() {
            if (!p.w_stationary) return;
            const int i = (int)threadIdx.x - 32;
            if (i >= TM) return;
            const int nb = level_begin(lvl + 1), ne = level_begin(lvl + 2);
            const int tmr2 = rows_per_tile(ne - nb, tiles_u, p.n_sms);
            const int tiles2 = ((ne - nb + tmr2 - 1) / tmr2) * tiles_u;
            if ((int)blockIdx.x >= tiles2 || i >= tmr2) return;
            const int row = nb + ((int)blockIdx.x / tiles_u) * tmr2 + i;
            int node = -1, l = 0, r = 0;
            if (row < ne) {
              node = chk(p.st, p.order[row], p.n);
              l = chk(p.st, p.left[node], p.n);
              r = chk(p.st, p.right[node], p.n);
            }
            s_node[i] = node; s_l[i] = l; s_r[i] = r;
          });
      if (!passed) return;
      TL_STAMP(trace, lvl, 2);
      ids_ahead = p.w_stationary != 0;
    }
  }
}

}  // namespace

int launch_forward_fp32(treelstm* ctx, int n, const int32_t* left, const int32_t* right,
                        const int32_t* token, float* h, float* c, const int32_t* order,
                        const int32_t* level_offset_dev, const int32_t* level_offset_host,
                        int n_levels_host, int flags, void* ws, const WsLayout& lay,
                        cudaStream_t stream) {
  char* base = static_cast<char*>(ws);
  FwdParams p;
  p.n = n; p.H = ctx->H; p.E = ctx->E; p.n_sms = ctx->sm_count; p.vocab = ctx->vocab;
  p.chk_counts = check_counters(ws, lay);
  p.left = left; p.right = right; p.token = token; p.order = order;
  p.level_offset = level_offset_dev;
  p.emb = ctx->emb; p.W = ctx->W; p.b = ctx->b;
  p.h = h; p.c = c;
  p.gates = (flags & TREELSTM_SAVE_FOR_BACKWARD) ? reinterpret_cast<float*>(base + lay.gates) : nullptr;
  p.st = reinterpret_cast<DevStatus*>(base + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  p.w_stationary = 0; p.a_row = 0; p.w_row = 0;
#ifdef TREELSTM_TRACE
  p.trace = reinterpret_cast<long long*>(base + lay.trace) + kTraceSlots * kTraceLevels;   // second table: the backward clears the first
  if (flags & TREELSTM_PERSISTENT)
    TL_CUDA(ctx, cudaMemsetAsync(p.trace, 0, sizeof(long long) * kTraceSlots * kTraceLevels, stream));
#endif
  const int tiles_u = (ctx->H + TU - 1) / TU;
  if (flags & TREELSTM_PERSISTENT) {
    // Resident W_h slice: 80 rows of w_row floats (w_row = 4 mod 32, so that the float4 reads of the
    // sixteen columns of a gate spread over all banks) next to the operand rows of one tile.
    const int K4 = (2 * ctx->H + 3) & ~3;
    p.a_row = K4 + 4;
    p.w_row = K4 + ((4 - K4 % 32) + 32) % 32;
    size_t a_bytes = sizeof(float) * TM * (size_t)p.a_row;
    if (a_bytes < sizeof(TileSmem)) a_bytes = sizeof(TileSmem);
    a_bytes = (a_bytes + 15) & ~(size_t)15;
    const size_t ids_bytes = 3 * TM * sizeof(int);
    const size_t smem_stat = a_bytes + sizeof(float) * 5 * TU * (size_t)p.w_row + sizeof(float) * 4 * TMS * 5 * TU + ids_bytes;
    size_t smem = sizeof(TileSmem) + ids_bytes;
    p.w_stationary = 0;
    int cap = ctx->opt.max_ctas > 0 ? ctx->opt.max_ctas : (1 << 30);
    if (smem_stat <= 216 * 1024 && ctx->sm_count >= tiles_u && cap >= tiles_u) {
      p.w_stationary = 1;
      smem = smem_stat;
    } else {
      p.a_row = p.w_row = 0;
    }
    TL_CUDA(ctx, cudaFuncSetAttribute(k_fwd_fp32_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    int per_sm = 0;
    TL_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fwd_fp32_persistent,
                                                               kThreads, smem));
    // Started under the single-CTA scheduler (see launch_forward_bf16 for the two ways to launch a
    // kernel with a grid barrier): the scheduler keeps its SM.
    const int single_max = ctx->opt.sched_single_cta_max < kSchedSingleMaxNodes ? ctx->opt.sched_single_cta_max : kSchedSingleMaxNodes;
    const bool overlap = ctx->opt.overlap_launch && n <= single_max && per_sm >= 1 && ctx->sm_count > 1;
    p.early_start = overlap ? 1 : 0;
    int grid = per_sm * (overlap ? ctx->sm_count - 1 : ctx->sm_count);
    const int want = ((n + TMS - 1) / TMS + 1) * tiles_u;   // never more CTAs than the widest level has tiles
    if (grid > want) grid = want;
    if (grid > cap) grid = cap;
    if (p.w_stationary) grid = grid / tiles_u * tiles_u;    // every CTA keeps one hidden-unit slice
    if (grid < 1) grid = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream;
    cudaLaunchAttribute attr;
    if (overlap) {
      attr.id = cudaLaunchAttributeProgrammaticStreamSerialization; attr.val.programmaticStreamSerializationAllowed = 1;
    } else {
      attr.id = cudaLaunchAttributeCooperative; attr.val.cooperative = 1;
    }
    cfg.attrs = &attr; cfg.numAttrs = 1;
    TL_CUDA(ctx, cudaLaunchKernelEx(&cfg, k_fwd_fp32_persistent, p));
    ctx->launches += 1;
    return TREELSTM_OK;
  }
  for (int lvl = 0; lvl < n_levels_host; ++lvl) {
    const int begin = level_offset_host[lvl], end = level_offset_host[lvl + 1];
    const int tmr = rows_per_tile(end - begin, tiles_u, p.n_sms);
    const int tiles = ((end - begin + tmr - 1) / tmr) * tiles_u;
    if (tiles <= 0) continue;
    k_fwd_fp32_level<<<tiles, kThreads, 0, stream>>>(p, begin, end, lvl == 0 ? 1 : 0);
    ctx->launches += 1;
  }
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

}  // namespace tl
