// The paper's other two recursive models on the same scheduler (Section 6.1: TreeRNN and RNTN next
// to TreeLSTM; Table 1 of Section 6.3 is measured on TreeRNN), fp32:
//
//   TreeRNN   p   = tanh(W^T [h_l ; h_r] + b)
//   RNTN      p_j = tanh([h_l ; h_r]^T V_j [h_l ; h_r] + (W^T [h_l ; h_r])_j + b_j)
//
// A leaf's state is its word vector (h = emb[token], embedding width = H); there is no cell state.
// Evaluation is the one of Figure 2 with all ready nodes of a wavefront at once (Section 2.2: the two
// child calls are independent).
//
// Both cells are one contraction per wavefront: the operand row of a node is [x (x) x ; x] with
// x = [h_l ; h_r] (TreeRNN: x alone), the weight matrix Wcat = [Vt ; W] with Vt[a * 2H + b][j] =
// V[j][a][b], re-packed once at create.  The products x_a * x_b are formed while a chunk of the
// contraction is staged in shared memory; nothing of the 4H^2-wide row is ever written out.
#include "common.cuh"

namespace tl {
namespace {

constexpr int RM = 32;        // nodes per tile
constexpr int RN = 64;        // hidden units per tile
constexpr int RK = 32;        // contraction chunk
constexpr int kThreads = 256;

struct RecParams {
  int n, H, cell, K, vocab;   // K: contraction length (2H, or 4H^2 + 2H)
  int* chk_counts;            // checked build: writes of h per node
  const int *left, *right, *token, *order, *level_offset;
  const float *emb, *Wcat, *b;
  float* h;
  DevStatus* st;
  long long wait_limit;
};

// rows [row_begin, row_end) of the ready order (level 0): the word vectors
__device__ void rec_leaves(const RecParams& p, int row_begin, int row_end, int gtid, int gthreads) {
  const int H = p.H;
  const long long total = (long long)(row_end - row_begin) * H;
  for (long long i = gtid; i < total; i += gthreads) {
    const int row = row_begin + (int)(i / H), u = (int)(i % H);
    const int node = chk(p.st, p.order[row], p.n);
    p.h[(size_t)node * H + u] = __ldg(p.emb + (size_t)chk(p.st, p.token[node], p.vocab) * H + u);
    count_write(p.chk_counts, node, 1);
  }
}

// One tile: rows [row0, row0 + RM) of the ready order (clipped to row_end) x hidden units
// [u0, u0 + RN).  smem: X[RM][2H + 1] (the children's states of every row), As[RM][RK + 1],
// Bs[RK][RN], node ids.  Thread (tx, ty), tx = tid % 16, ty = tid / 16: rows ty and ty + 16, units
// u0 + tx + 16 q for q = 0..3.
__device__ void rec_tile(const RecParams& p, int row0, int row_end, int u0, float* smem) {
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int H = p.H, K2 = 2 * H, xs = K2 + 1;
  const int KQ = p.cell == TREELSTM_CELL_RNTN ? K2 * K2 : 0;    // length of the quadratic part
  float* X = smem;
  float* As = X + RM * xs;
  float* Bs = As + RM * (RK + 1);
  int* s_node = reinterpret_cast<int*>(Bs + RK * RN);
  __syncthreads();   // the previous tile's readers are done
  for (int i = tid; i < RM; i += kThreads) s_node[i] = row0 + i < row_end ? chk(p.st, p.order[row0 + i], p.n) : -1;
  __syncthreads();
  for (int e = tid; e < RM * K2; e += kThreads) {
    const int i = e / K2, k = e - i * K2;
    const int node = s_node[i];
    float v = 0.f;
    if (node >= 0) {
      const int child = chk(p.st, k < H ? p.left[node] : p.right[node], p.n);
      v = __ldcg(p.h + (size_t)child * H + (k < H ? k : k - H));
    }
    X[i * xs + k] = v;
  }
  __syncthreads();
  float acc[2][4] = {};
  for (int k0 = 0; k0 < p.K; k0 += RK) {
    // operand chunk: products of two entries of x for the tensor part, x itself for the linear part
    for (int e = tid; e < RM * RK; e += kThreads) {
      const int i = e / RK, kk = e - i * RK, k = k0 + kk;
      float v = 0.f;
      if (k < KQ) {
        const int a = k / K2, bb = k - a * K2;
        v = X[i * xs + a] * X[i * xs + bb];
      } else if (k < p.K) {
        v = X[i * xs + (k - KQ)];
      }
      As[i * (RK + 1) + kk] = v;
    }
    for (int e = tid; e < RK * RN; e += kThreads) {
      const int kk = e / RN, j = e - kk * RN, k = k0 + kk;
      Bs[e] = (k < p.K && u0 + j < H) ? __ldg(p.Wcat + (size_t)k * H + u0 + j) : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < RK; ++kk) {
      const float a0 = As[ty * (RK + 1) + kk], a1 = As[(ty + 16) * (RK + 1) + kk];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float w = Bs[kk * RN + tx + 16 * q];
        acc[0][q] = fmaf(a0, w, acc[0][q]);
        acc[1][q] = fmaf(a1, w, acc[1][q]);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    const int node = s_node[ty + 16 * r];
    if (node < 0) continue;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int u = u0 + tx + 16 * q;
      if (u < H) {
        p.h[(size_t)node * H + u] = tanhf(acc[r][q] + __ldg(p.b + u));
        count_write(p.chk_counts, node, 1);
      }
    }
  }
}

__global__ void k_rec_leaves(RecParams p, int row_begin, int row_end) {
  rec_leaves(p, row_begin, row_end, blockIdx.x * blockDim.x + threadIdx.x, gridDim.x * blockDim.x);
}

__global__ void __launch_bounds__(kThreads) k_rec_level(RecParams p, int row_begin, int row_end) {
  extern __shared__ float rec_smem[];
  const int tiles_u = (p.H + RN - 1) / RN;
  rec_tile(p, row_begin + (blockIdx.x / tiles_u) * RM, row_end, (blockIdx.x % tiles_u) * RN, rec_smem);
}

// All wavefronts in one cooperative launch; the bounded grid barrier separates them.
__global__ void __launch_bounds__(kThreads) k_rec_persistent(RecParams p) {
  extern __shared__ float rec_smem[];
  __shared__ int s_flag;
  if (ld_volatile(&p.st->status) != 0) return;
  const int n_levels = p.st->n_levels;
  const int tiles_u = (p.H + RN - 1) / RN;
  for (int lvl = 0; lvl < n_levels; ++lvl) {
    const int begin = p.level_offset[lvl], end = p.level_offset[lvl + 1];
    if (lvl == 0) {
      rec_leaves(p, begin, end, blockIdx.x * kThreads + threadIdx.x, gridDim.x * kThreads);
    } else {
      const int tiles = ((end - begin + RM - 1) / RM) * tiles_u;
      for (int t = blockIdx.x; t < tiles; t += gridDim.x)
        rec_tile(p, begin + (t / tiles_u) * RM, end, (t % tiles_u) * RN, rec_smem);
    }
    if (lvl + 1 < n_levels && !grid_barrier(p.st, (unsigned)(lvl + 1) * gridDim.x, p.wait_limit, &s_flag)) return;
  }
}

// Wcat = [Vt ; W]: Vt[(a * 2H + b)][j] = V[j][a][b] (RNTN only), then the 2H rows of W.
__global__ void k_rec_pack(int H, int cell, const float* W, const float* V, float* Wcat) {
  const size_t K2 = 2 * (size_t)H, KQ = cell == TREELSTM_CELL_RNTN ? K2 * K2 : 0;
  const size_t total = (KQ + K2) * H, stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += stride) {
    const size_t k = i / H, j = i % H;
    Wcat[i] = k < KQ ? V[j * KQ + k] : W[(k - KQ) * H + j];
  }
}

size_t rec_smem_bytes(int H) {
  return sizeof(float) * ((size_t)RM * (2 * H + 1) + RM * (RK + 1) + RK * RN) + sizeof(int) * RM;
}

}  // namespace

int pack_weights_rec(treelstm* ctx, const float* W, const float* V, cudaStream_t stream) {
  k_rec_pack<<<512, 256, 0, stream>>>(ctx->H, ctx->cell, W, V, ctx->Wcat);
  TL_CUDA(ctx, cudaGetLastError());
  const size_t smem = rec_smem_bytes(ctx->H);
  if (smem > 200 * 1024) return TREELSTM_ERR_UNSUPPORTED;
  TL_CUDA(ctx, cudaFuncSetAttribute(k_rec_level, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  TL_CUDA(ctx, cudaFuncSetAttribute(k_rec_persistent, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  return TREELSTM_OK;
}

int launch_forward_rec(treelstm* ctx, int n, const int32_t* left, const int32_t* right, const int32_t* token,
                       float* h, const int32_t* order, const int32_t* level_offset_dev,
                       const int32_t* level_offset_host, int n_levels_host, int flags, void* ws,
                       const WsLayout& lay, cudaStream_t stream) {
  RecParams p;
  p.n = n; p.H = ctx->H; p.cell = ctx->cell; p.vocab = ctx->vocab;
  p.chk_counts = check_counters(ws, lay);
  p.K = ctx->cell == TREELSTM_CELL_RNTN ? 4 * ctx->H * ctx->H + 2 * ctx->H : 2 * ctx->H;
  p.left = left; p.right = right; p.token = token; p.order = order; p.level_offset = level_offset_dev;
  p.emb = ctx->emb; p.Wcat = ctx->Wcat; p.b = ctx->b;
  p.h = h;
  p.st = reinterpret_cast<DevStatus*>(static_cast<char*>(ws) + lay.status);
  p.wait_limit = ctx->opt.wait_limit_kcycles * 1024;
  const size_t smem = rec_smem_bytes(ctx->H);
  const int tiles_u = (ctx->H + RN - 1) / RN;
  if (flags & TREELSTM_PERSISTENT) {
    int per_sm = 0;
    TL_CUDA(ctx, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_rec_persistent, kThreads, smem));
    if (per_sm < 1) return TREELSTM_ERR_UNSUPPORTED;
    int grid = per_sm * ctx->sm_count;
    const int want = ((n + RM - 1) / RM + 1) * tiles_u;   // never more CTAs than the widest wavefront has tiles
    if (grid > want) grid = want;
    if (ctx->opt.max_ctas > 0 && grid > ctx->opt.max_ctas) grid = ctx->opt.max_ctas;
    if (grid < 1) grid = 1;
    void* args[] = {&p};
    TL_CUDA(ctx, cudaLaunchCooperativeKernel((void*)k_rec_persistent, dim3(grid), dim3(kThreads), args, smem, stream));
    ctx->launches += 1;
    return TREELSTM_OK;
  }
  for (int lvl = 0; lvl < n_levels_host; ++lvl) {
    const int begin = level_offset_host[lvl], end = level_offset_host[lvl + 1];
    if (end <= begin) continue;
    if (lvl == 0) {
      const long long total = (long long)(end - begin) * ctx->H;
      const int blocks = (int)((total + 255) / 256 < 2048 ? (total + 255) / 256 : 2048);
      k_rec_leaves<<<blocks, 256, 0, stream>>>(p, begin, end);
    } else {
      const int tiles = ((end - begin + RM - 1) / RM) * tiles_u;
      k_rec_level<<<tiles, kThreads, smem, stream>>>(p, begin, end);
    }
    ctx->launches += 1;
  }
  TL_CUDA(ctx, cudaGetLastError());
  return TREELSTM_OK;
}

}  // namespace tl
