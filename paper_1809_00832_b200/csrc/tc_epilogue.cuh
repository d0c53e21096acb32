// The epilogue of one tile, shared by the grid-wide wavefront kernel (gemm_tc.cu) and the sub-forest
// kernel (subforest_tc.cu): drain the accumulator from tensor memory, finish the TreeLSTM cell
// (c = i*u + f_l*c_l + f_r*c_r, h = o*tanh(c); a leaf has no children and no forget gates), and
// deliver the state - fp32 h and c at the node id, bf16 h and fp32 c into the operand row of the
// node's caller.
//
// 256 epilogue threads: thread = tile row r (tensor-memory lane) x half e; set e takes hidden
// units [4e, 4e + 4) of every unit group of the tile.  A staging row per tile row in shared memory
// holds first the children's cell states (fetched by cp.async while the MMAs run), then the new c
// and h: all epilogue threads then copy whole row segments out, several lanes per row, so that a
// warp store covers a few full lines instead of 32 scattered 16-byte pieces.
#pragma once

#include "tc_ptx.cuh"

namespace tl {

struct EpiTile {
  // the tile
  bool leaf;
  int G, gcols, ncols, nt;      // unit groups, packed columns per group, columns in use, column tile (units of G groups)
  int row, node, slot;          // this thread's operand row, its node and delivery slot (2 * pos(caller) + side, -1: root)
  bool valid;                   // the row belongs to the tile
  bool allow_staged_out;        // copy the outputs out through the staging rows (else straight from registers)
  // the thread
  int r, e, quad;
  // shared memory: staging rows of (1 << crow_shift) bytes, second half at chunk index `half`
  uint32_t cstage_addr;
  unsigned char* cstage_ptr;
  uint32_t crow_shift;
  int half;
  int *s_rownode, *s_rowslot;
  // synchronisation
  uint32_t tmem_acc;            // tensor-memory address of the accumulator stage
  uint32_t tfull, tempty, epi_bar, acc_phase;
  const float* bias;            // packed bias of the tile's first column, this thread's half
  long long* stamp = nullptr;   // trace builds: three cycle stamps of this tile (accumulator ready, cells done, tile left)
};
#ifdef TREELSTM_TRACE
#define TL_TILE_STAMP(t, k) do { if ((t).stamp) (t).stamp[k] = clock64(); } while (0)
#else
#define TL_TILE_STAMP(t, k) do { } while (0)
#endif

// between_fn runs after the cell updates and before the accumulator is handed back (the callers
// fetch row data of their next tile there).
template <class BetweenFn>
__device__ __forceinline__ void epilogue_tile(const TcParams& p, const EpiTile& t, uint32_t& epi_phase, bool& alive,
                                              volatile int* s_abort, BetweenFn between_fn) {
  const int H = p.H, Hp = p.Hp, G = t.G, r = t.r, e = t.e, nt = t.nt, gcols = t.gcols;
  const bool leaf = t.leaf, valid = t.valid;
  const int node = t.node, slot = t.slot;
  const bool vec = (H % 4) == 0;
  const float* crow = p.cin + (size_t)t.row * 2 * H;   // [c_l | c_r] of the node at this position
  const bool full_slice = vec && (nt + 1) * G * 8 <= H;   // no padded unit among the tile's columns
  const bool staged = !leaf && full_slice;
  const bool staged_out = full_slice && p.gates == nullptr && t.allow_staged_out;
  const int half = t.half;
  const uint32_t my_c = t.cstage_addr + ((uint32_t)r << t.crow_shift);
  unsigned char* mine = t.cstage_ptr + ((size_t)r << t.crow_shift);
  if (staged) {   // the children's cell states of this thread's row, while the MMAs run
    const float* sl = crow + nt * G * 8;
    const float* sr = sl + H;
    const uint32_t nb = valid ? 16u : 0u;
    for (int ch = e; ch < 2 * G; ch += 2) {
      cp_async16(my_c + (uint32_t)((ch ^ (r & 7)) << 4), sl + ch * 4, nb);
      cp_async16(my_c + (uint32_t)(((half + ch) ^ (r & 7)) << 4), sr + ch * 4, nb);
    }
  }
  const float* bias = t.bias;
  const int ngates = leaf ? 3 : 5;
  float4 bnext[5];
#pragma unroll
  for (int q = 0; q < 5; ++q)
    if (q < ngates) bnext[q] = __ldg(reinterpret_cast<const float4*>(bias + 8 * q));
  if (!mbar_wait(t.tfull, t.acc_phase, s_abort, p.wait_limit, p.st)) alive = false;
  alive = __all_sync(kFullMask, alive);
  asm volatile("cp.async.wait_all;" ::: "memory");
  if (!alive) return;
  TL_TILE_STAMP(t, 0);
  tc_fence_after();
  const uint32_t taddr = t.tmem_acc + ((uint32_t)(t.quad * 32) << 16) + 4u * e;
  // the tensor-memory loads of group g + 1 are in flight while group g is computed
  uint32_t vbuf[2][20];
  auto load_group = [&](int g, uint32_t* v) {
    const uint32_t col0 = (uint32_t)(g * gcols);
    if (leaf) {
#pragma unroll
      for (int q = 0; q < 3; ++q) tmem_ld4(taddr + col0 + 8 * q, v + 4 * q);
    } else {
#pragma unroll
      for (int q = 0; q < 5; ++q) tmem_ld4(taddr + col0 + 8 * q, v + 4 * q);
    }
  };
  load_group(0, vbuf[0]);
#pragma unroll
  for (int g = 0; g < kMaxG; ++g) {
    if (g >= G) break;
    uint32_t* v = vbuf[g & 1];
    float4 bcur[5];
#pragma unroll
    for (int q = 0; q < 5; ++q) bcur[q] = bnext[q];
    tmem_ld_wait();
    if (g + 1 < G) {
      load_group(g + 1, vbuf[(g + 1) & 1]);
#pragma unroll
      for (int q = 0; q < 5; ++q)
        if (q < ngates) bnext[q] = __ldg(reinterpret_cast<const float4*>(bias + (g + 1) * gcols + 8 * q));
    }
    if (valid) {
      const int u0 = (nt * G + g) * 8 + 4 * e;
      const int count = min(4, H - u0);     // real (unpadded) units among these four
      float cl[4] = {}, cr[4] = {}, hv[4], cv[4], gi[4], gfl[4], gfr[4], go[4], gu[4];
      if (staged) {
        const float4 a = *reinterpret_cast<const float4*>(mine + (((2 * g + e) ^ (r & 7)) << 4));
        const float4 b = *reinterpret_cast<const float4*>(mine + (((half + 2 * g + e) ^ (r & 7)) << 4));
        cl[0] = a.x; cl[1] = a.y; cl[2] = a.z; cl[3] = a.w;
        cr[0] = b.x; cr[1] = b.y; cr[2] = b.z; cr[3] = b.w;
      } else if (!leaf && count > 0) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          cl[j] = j < count ? __ldcg(crow + u0 + j) : 0.f;
          cr[j] = j < count ? __ldcg(crow + H + u0 + j) : 0.f;
        }
      }
      const float* bq = reinterpret_cast<const float*>(bcur);
      // every step over all four units before the next one: twenty independent activations in flight
      if (leaf) {
        float z[12];
#pragma unroll
        for (int j = 0; j < 12; ++j) z[j] = __uint_as_float(v[j]) + bq[j];
#pragma unroll
        for (int j = 0; j < 4; ++j) { gi[j] = act_sigmoid(z[j]); go[j] = act_sigmoid(z[4 + j]); gu[j] = act_tanh(z[8 + j]); }
#pragma unroll
        for (int j = 0; j < 4; ++j) { gfl[j] = gfr[j] = 0.f; cv[j] = gi[j] * gu[j]; }
      } else {
        float z[20];
#pragma unroll
        for (int j = 0; j < 20; ++j) z[j] = __uint_as_float(v[j]) + bq[j];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          gi[j] = act_sigmoid(z[j]); gfl[j] = act_sigmoid(z[4 + j]); gfr[j] = act_sigmoid(z[8 + j]);
          go[j] = act_sigmoid(z[12 + j]); gu[j] = act_tanh(z[16 + j]);
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) cv[j] = gi[j] * gu[j] + gfl[j] * cl[j] + gfr[j] * cr[j];
      }
      float tcv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) tcv[j] = act_tanh(cv[j]);
#pragma unroll
      for (int j = 0; j < 4; ++j) hv[j] = go[j] * tcv[j];
      if (staged_out) {
        *reinterpret_cast<float4*>(mine + (((2 * g + e) ^ (r & 7)) << 4)) = make_float4(cv[0], cv[1], cv[2], cv[3]);
        *reinterpret_cast<float4*>(mine + (((half + 2 * g + e) ^ (r & 7)) << 4)) = make_float4(hv[0], hv[1], hv[2], hv[3]);
      } else {
        if (slot >= 0) {
          // hand the state to the caller: bf16 h into its operand row (padded units as 0),
          // fp32 c next to it
          uint32_t packed[2];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const float lo = 2 * j < count ? hv[2 * j] : 0.f, hi = 2 * j + 1 < count ? hv[2 * j + 1] : 0.f;
            __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
            packed[j] = *reinterpret_cast<uint32_t*>(&b2);
          }
          *reinterpret_cast<uint2*>(p.ain + (size_t)slot * Hp + u0) = make_uint2(packed[0], packed[1]);
          if (count > 0) st_row4(p.cin + (size_t)slot * H + u0, vec, count, cv);
          count_write(p.chk_counts ? p.chk_counts + p.n : nullptr, slot >> 1, count);
          count_write(p.chk_counts ? p.chk_counts + 2 * p.n : nullptr, slot >> 1, count);
        }
        if (count > 0) {
          count_write(p.chk_counts, node, count);
          st_row4(p.h + (size_t)node * H + u0, vec, count, hv);
          st_row4(p.c + (size_t)node * H + u0, vec, count, cv);
          if (p.gates) {
            float* gp = p.gates + (size_t)node * 5 * H + u0;
            st_row4(gp, vec, count, gi);
            st_row4(gp + H, vec, count, gfl);
            st_row4(gp + 2 * H, vec, count, gfr);
            st_row4(gp + 3 * H, vec, count, go);
            st_row4(gp + 4 * H, vec, count, gu);
          }
        }
      }
    }
  }
  TL_TILE_STAMP(t, 1);
  between_fn();
  tc_fence_before();
  mbar_arrive(t.tempty);                       // accumulator stage may be overwritten
  if (staged_out) {
    if (e == 0) { t.s_rownode[r] = valid ? node : -1; t.s_rowslot[r] = slot; }
    mbar_arrive(t.epi_bar);
    bool ok = mbar_wait(t.epi_bar, epi_phase, s_abort, p.wait_limit, p.st);
    epi_phase ^= 1;
    if (ok) {
      const int et = e * BM + r, cpr = 2 * G;           // 16-byte chunks (4 units) per row
      const int lcpr = (cpr & (cpr - 1)) == 0 ? 31 - __clz(cpr) : -1;   // a shift where 2 G is a power of two
      for (int idx = et; idx < BM * cpr; idx += 2 * BM) {
        const int ro = lcpr >= 0 ? idx >> lcpr : idx / cpr, ch = idx - ro * cpr;
        const int node_o = t.s_rownode[ro];
        if (node_o < 0) continue;
        const unsigned char* src = t.cstage_ptr + ((size_t)ro << t.crow_shift);
        const float4 c4 = *reinterpret_cast<const float4*>(src + ((ch ^ (ro & 7)) << 4));
        const float4 h4 = *reinterpret_cast<const float4*>(src + (((half + ch) ^ (ro & 7)) << 4));
        const int uo = nt * G * 8 + 4 * ch;
        *reinterpret_cast<float4*>(p.h + (size_t)node_o * H + uo) = h4;
        *reinterpret_cast<float4*>(p.c + (size_t)node_o * H + uo) = c4;
        count_write(p.chk_counts, node_o, 4);
        const int slot_o = t.s_rowslot[ro];
        if (slot_o >= 0) {
          count_write(p.chk_counts ? p.chk_counts + p.n : nullptr, slot_o >> 1, 4);
          count_write(p.chk_counts ? p.chk_counts + 2 * p.n : nullptr, slot_o >> 1, 4);
          *reinterpret_cast<float4*>(p.cin + (size_t)slot_o * H + uo) = c4;
          __nv_bfloat162 lo = __floats2bfloat162_rn(h4.x, h4.y), hi = __floats2bfloat162_rn(h4.z, h4.w);
          *reinterpret_cast<uint2*>(p.ain + (size_t)slot_o * Hp + uo) =
              make_uint2(*reinterpret_cast<uint32_t*>(&lo), *reinterpret_cast<uint32_t*>(&hi));
        }
      }
    }
    // the staging rows are reused by the next tile's loads of the children's cell states
    mbar_arrive(t.epi_bar);
    ok = mbar_wait(t.epi_bar, epi_phase, s_abort, p.wait_limit, p.st) && ok;
    epi_phase ^= 1;
    if (!ok) alive = false;
  }
  TL_TILE_STAMP(t, 2);
}

}  // namespace tl
