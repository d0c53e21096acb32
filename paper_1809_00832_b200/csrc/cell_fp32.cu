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
  int n, H, E, n_sms;
  const int *left, *right, *token, *order, *level_offset;
  const float *emb, *W, *b;
  float *h, *c, *gates;
  DevStatus* st;
  long long wait_limit;
};

__device__ __forceinline__ float sigmoidf_acc(float x) { return 1.0f / (1.0f + expf(-x)); }

struct TileSmem {
  float A[2][TM][KC + 1];
  float W[2][KC][5 * TU];
  int node[TM], l[TM], r[TM];
};

// Rows per tile of a wavefront of `rows` nodes: a level-uniform choice.
__host__ __device__ inline int rows_per_tile(int rows, int tiles_u, int n_sms) {
  return ((rows + TM - 1) / TM) * tiles_u >= n_sms ? TM : TMS;
}

// One tile: rows [row0, row0 + TM) of the ready order (clipped to row_end), hidden units
// [u0, u0 + TU).  `leaf` selects x = emb[token] with W rows [0, E) and gates i, o, u only.
// The next K chunk is fetched into registers while the current one is multiplied out of shared
// memory (two buffers, one CTA barrier per chunk).
template <int TM>
__device__ void fp32_tile(const FwdParams& p, int row0, int row_end, int u0, bool leaf,
                          TileSmem& s) {
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
      node = p.order[row];
      l = leaf ? p.token[node] : p.left[node];
      r = leaf ? 0 : p.right[node];
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
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < kALoads; ++j) {
      const int e = tid + j * kThreads, i = e / KC, k = k0 + e % KC;
      float v = 0.f;
      if (s.node[i] >= 0 && k < K) {
        if (leaf) v = __ldg(p.emb + (size_t)s.l[i] * E + k);
        else v = k < H ? __ldcg(p.h + (size_t)s.l[i] * H + k) : __ldcg(p.h + (size_t)s.r[i] * H + (k - H));
      }
      ra[j] = v;
    }
#pragma unroll
    for (int j = 0; j < kWLoads; ++j) {
      const int e = tid + j * kThreads, kk = e / (5 * TU), g = (e % (5 * TU)) / TU, uu = e % TU, k = k0 + kk;
      float v = 0.f;
      if (k < K && u0 + uu < H && !(leaf && (g == 1 || g == 2)))
        v = __ldg(Wk + (size_t)k * 5 * H + g * H + u0 + uu);
      rw[j] = v;
    }
  };
  auto stash = [&](int buf) {
#pragma unroll
    for (int j = 0; j < kALoads; ++j) {
      const int e = tid + j * kThreads;
      s.A[buf][e / KC][e % KC] = ra[j];
    }
#pragma unroll
    for (int j = 0; j < kWLoads; ++j) {
      const int e = tid + j * kThreads;
      s.W[buf][e / (5 * TU)][e % (5 * TU)] = rw[j];
    }
  };
  fetch(0);
  stash(0);
  __syncthreads();
  const int chunks = (K + KC - 1) / KC;
  for (int cidx = 0; cidx < chunks; ++cidx) {
    const int buf = cidx & 1;
    if (cidx + 1 < chunks) fetch((cidx + 1) * KC);
#pragma unroll
    for (int kk = 0; kk < KC; ++kk) {
      float a[RPT], w[5];
#pragma unroll
      for (int i = 0; i < RPT; ++i) a[i] = s.A[buf][ty * RPT + i][kk];
#pragma unroll
      for (int g = 0; g < 5; ++g) w[g] = s.W[buf][kk][g * TU + tx];
#pragma unroll
      for (int i = 0; i < RPT; ++i)
#pragma unroll
        for (int g = 0; g < 5; ++g) acc[i][g] = fmaf(a[i], w[g], acc[i][g]);
    }
    if (cidx + 1 < chunks) stash(buf ^ 1);
    __syncthreads();
  }

  const int u = u0 + tx;
  if (u >= H) return;
  float bias[5];
#pragma unroll
  for (int g = 0; g < 5; ++g) bias[g] = __ldg(p.b + g * H + u);
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
    if (p.gates) {
      float* g = p.gates + (size_t)node * 5 * H + u;
      g[0] = gi; g[H] = gfl; g[2 * H] = gfr; g[3 * H] = go; g[4 * H] = gu;
    }
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
__global__ void __launch_bounds__(kThreads)
k_fwd_fp32_persistent(FwdParams p) {
  __shared__ TileSmem s;
  __shared__ int s_flag;
  if (ld_volatile(&p.st->status) != 0) return;
  const int n_levels = p.st->n_levels;
  const int tiles_u = (p.H + TU - 1) / TU;
  for (int lvl = 0; lvl < n_levels; ++lvl) {
    const int begin = p.level_offset[lvl], end = p.level_offset[lvl + 1];
    const int tmr = rows_per_tile(end - begin, tiles_u, p.n_sms);
    const int tiles = ((end - begin + tmr - 1) / tmr) * tiles_u;
    for (int t = blockIdx.x; t < tiles; t += gridDim.x) {
      if (tmr == TM) fp32_tile<TM>(p, begin + (t / tiles_u) * TM, end, (t % tiles_u) * TU, lvl == 0, s);
      else fp32_tile<TMS>(p, begin + (t / tiles_u) * TMS, end, (t % tiles_u) * TU, lvl == 0, s);
    }
    if (lvl + 1 < n_levels &&
        !grid_barrier(p.st, (unsigned)(lvl + 1) * gridDim.x, p.wait_limit, &s_flag))
      return;
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
  p.n = n; p.H = ctx->H; p.E = ctx->E; p.n_sms = ctx->sm_count;
  p.left = left; p.right = right; p.token = token; p.order = order;
  p.level_offset = level_offset_dev;
  p.emb = ctx->emb; p.W = ctx->W; p.b = ctx->b;
  p.h = h; p.c = c;
  p.gates = (flags & TREELSTM_SAVE_FOR_BACKWARD) ? reinterpret_cast<float*>(base + lay.gates) : nullptr;
  p.st = reinterpret_cast<DevStatus*>(base + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  const int tiles_u = (ctx->H + TU - 1) / TU;
  if (flags & TREELSTM_PERSISTENT) {
    int per_sm = 0;
    TL_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_fwd_fp32_persistent,
                                                               kThreads, 0));
    int grid = per_sm * ctx->sm_count;
    const int want = ((n + TMS - 1) / TMS + 1) * tiles_u;   // never more CTAs than the widest level has tiles
    if (grid > want) grid = want;
    if (ctx->opt.max_ctas > 0 && grid > ctx->opt.max_ctas) grid = ctx->opt.max_ctas;
    if (grid < 1) grid = 1;
    void* args[] = {&p};
    TL_CUDA(ctx, cudaLaunchCooperativeKernel((void*)k_fwd_fp32_persistent, dim3(grid), dim3(kThreads),
                                             args, 0, stream));
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
