// Thread-block CLUSTERS for the three vocabulary-wide stages of a round, ONE launch each:
//   k_ensemble_req : Algorithm 1 steps 6-7   (softmax of the m drafter rows, weighted average, draw)
//                    one cluster per request
//   k_verify_req   : Sec. 3 item 3           (target softmax, sequential acceptance, residual / bonus draw)
//                    one cluster per (request, position): the softmax of the G + 1 target rows runs on all of
//                    them at once; the cluster that finishes a request last (a ticket) takes its acceptance
//                    prefix and draws the replacement / bonus token
//   k_update_req   : Sec. 4.1, App. B        (deviation of every drafter over the verified positions, window
//                                             push, policy, cache commit)
//                    one cluster per (request, verified position); the last one of a request runs the policy
// No spin-wait anywhere: the vocabulary is cut into one contiguous slice per CTA of the cluster; every
// vocabulary-wide quantity (row maxima, integer mass sums, per-slice masses, deviation sums) is exchanged
// through distributed shared memory and ordered by the hardware cluster barrier; clusters of one request meet
// through a ticket counter (taken after a fence, reset by the last arriver, so no memset is needed).  A row is read from HBM once; the later passes of the exact
// softmax (maximum -> integer sum of masses -> quotient) re-read the CTA's own slice, which L1/L2 still hold.
// Loads are 128-bit where the row pitch allows, reductions are warp shuffles.  All decision arithmetic is
// the order-independent specification of exact_math.cuh, so the results do not depend on the cluster size.
#pragma once
#include <cooperative_groups.h>

#include "decide_kernels.cuh"
#include "exact_math.cuh"
#include "forward_kernels.cuh"

namespace tabed {

namespace cg = cooperative_groups;

constexpr int kReqThreads = 512;
constexpr int kReqWarps = kReqThreads / 32;
constexpr int kReqMaxCluster = 16;          // CTAs per cluster (16 needs the non-portable opt-in, 8 is portable)
constexpr int kReqMaxRows = 17;             // rows of one request handled together: gamma + 1 <= 17, m <= 8
constexpr int kReqStep = kReqThreads * 4;   // vocabulary elements one pass of the CTA covers
constexpr int kReqMaxWidth = 4;             // candidates per depth of a token tree

struct ReqCtx {
  unsigned CS, rank;
  int tid, lane, warp;
  int v_lo, v_hi;                           // this CTA's slice of the vocabulary
};

__device__ __forceinline__ void req_ld4(const float* __restrict__ row, int v, int v_hi, bool vec, float fill, float (&x)[4]) {
  if (vec && v + 4 <= v_hi) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(row + v));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) x[j] = (v + j < v_hi) ? __ldg(row + v + j) : fill;
  }
}
// coherent variant for data this very kernel has written (p)
__device__ __forceinline__ void req_ld4_rw(const float* row, int v, int v_hi, bool vec, float fill, float (&x)[4]) {
  if (vec && v + 4 <= v_hi) {
    const float4 a = *reinterpret_cast<const float4*>(row + v);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) x[j] = (v + j < v_hi) ? row[v + j] : fill;
  }
}
__device__ __forceinline__ void req_st4(float* __restrict__ row, int v, int v_hi, bool vec, const float (&x)[4]) {
  if (vec && v + 4 <= v_hi) {
    *reinterpret_cast<float4*>(row + v) = make_float4(x[0], x[1], x[2], x[3]);
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) if (v + j < v_hi) row[v + j] = x[j];
  }
}
__device__ __forceinline__ bool req_vec_ok(const void* base, long long pitch_elems) {
  return (pitch_elems & 3) == 0 && (reinterpret_cast<uintptr_t>(base) & 15) == 0;
}

struct ReqBest { float val; int idx; };
__device__ __forceinline__ void best_merge(ReqBest& a, const ReqBest& o) {
  if (o.val > a.val || (o.val == a.val && o.idx < a.idx)) a = o;
}

// Shared state of the softmax passes: per-warp partials, then one entry per (CTA of the cluster, row).
struct ReqShared {
  float red_f[kReqWarps][kReqMaxRows];
  unsigned long long red_u[kReqWarps][kReqMaxRows];
  ReqBest red_b[kReqWarps][kReqMaxRows];
  float all_max[kReqMaxCluster][kReqMaxRows];
  unsigned long long all_sum[kReqMaxCluster][kReqMaxRows];
  ReqBest all_best[kReqMaxCluster][kReqMaxRows];
  unsigned long long all_mass[4][kReqMaxCluster];
  unsigned long long scan[kReqWarps];
  unsigned long long scan2[kReqWarps];
  unsigned long long bc_mass[kReqMaxWidth];        // token and mass of candidate c, told to every CTA by the one that drew it
  int bc_tok[kReqMaxWidth];
  int ok[kReqMaxRows];
  int result;
  float par[3][kMaxInputs];                        // per-row scalars of a pass (maximum, normaliser, weight)
};

// Row maxima of `rows` rows (row i at base + i * pitch) over this CTA's slice, gathered over the cluster:
// afterwards S.all_max[r][i] holds CTA r's maximum of row i in every CTA.  Four rows' loads are in flight together.
// ebuf (optional, shared memory, row pitch epitch floats): the CTA's slice of every row is kept there, so that the later
// passes of the exact softmax neither go back to global memory nor take an exponential twice.
__device__ __forceinline__ void req_row_maxima(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, const float* __restrict__ base,
                                               long long pitch, int rows, bool vec, float* ebuf = nullptr, int epitch = 0) {
#pragma unroll 1
  for (int i0 = 0; i0 < rows; i0 += 4) {
    float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll 1
    for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
      float x[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + j < rows) req_ld4(base + (long long)(i0 + j) * pitch, v, c.v_hi, vec, -INFINITY, x[j]);
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (i0 + j < rows) {
          mx[j] = fmaxf(fmaxf(mx[j], fmaxf(x[j][0], x[j][1])), fmaxf(x[j][2], x[j][3]));
          if (ebuf) *reinterpret_cast<float4*>(ebuf + (size_t)(i0 + j) * epitch + (v - c.v_lo)) = make_float4(x[j][0], x[j][1], x[j][2], x[j][3]);
        }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float w = warp_max_f32(mx[j]);
      if (c.lane == 0 && i0 + j < rows) S.red_f[c.warp][i0 + j] = w;
    }
  }
  __syncthreads();
  if (c.tid < rows) {
    float v = S.red_f[0][c.tid];
#pragma unroll
    for (int w = 1; w < kReqWarps; ++w) v = fmaxf(v, S.red_f[w][c.tid]);
    for (unsigned r = 0; r < c.CS; ++r) cluster.map_shared_rank(&S.all_max[0][0], r)[c.rank * kReqMaxRows + c.tid] = v;
  }
  cluster.sync();
}
__device__ __forceinline__ float req_max_of(const ReqCtx& c, const ReqShared& S, int row) {
  float v = S.all_max[0][row];
  for (unsigned r = 1; r < c.CS; ++r) v = fmaxf(v, S.all_max[r][row]);
  return v;
}

// Integer sums of the exp masses of the rows (softmax normalisers), gathered over the cluster.
// With ebuf: reads the logits left there by req_row_maxima and leaves the exponentials in their place.
__device__ __forceinline__ void req_row_sums(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, const float* __restrict__ base,
                                             long long pitch, int rows, bool vec, float* ebuf = nullptr, int epitch = 0) {
#pragma unroll 1
  for (int i0 = 0; i0 < rows; i0 += 2) {
    unsigned long long sm[2] = {0ull, 0ull};
    float mx[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) mx[j] = (i0 + j < rows) ? req_max_of(c, S, i0 + j) : 0.0f;
#pragma unroll 1
    for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
      float x[2][4];
#pragma unroll
      for (int j = 0; j < 2; ++j)
        if (i0 + j < rows) {
          if (ebuf) {
            const float4 t = *reinterpret_cast<const float4*>(ebuf + (size_t)(i0 + j) * epitch + (v - c.v_lo));
            x[j][0] = t.x; x[j][1] = t.y; x[j][2] = t.z; x[j][3] = t.w;
          } else {
            req_ld4(base + (long long)(i0 + j) * pitch, v, c.v_hi, vec, -INFINITY, x[j]);
          }
        }
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        if (i0 + j >= rows) continue;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          x[j][e] = (v + e < c.v_hi) ? xexp(__fsub_rn(x[j][e], mx[j])) : 0.0f;
          if (v + e < c.v_hi) sm[j] += mass_of(x[j][e]);
        }
        if (ebuf) *reinterpret_cast<float4*>(ebuf + (size_t)(i0 + j) * epitch + (v - c.v_lo)) = make_float4(x[j][0], x[j][1], x[j][2], x[j][3]);
      }
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const unsigned long long w = warp_sum_u64(sm[j]);
      if (c.lane == 0 && i0 + j < rows) S.red_u[c.warp][i0 + j] = w;
    }
  }
  __syncthreads();
  if (c.tid < rows) {
    unsigned long long v = 0;
#pragma unroll
    for (int w = 0; w < kReqWarps; ++w) v += S.red_u[w][c.tid];
    for (unsigned r = 0; r < c.CS; ++r) cluster.map_shared_rank(&S.all_sum[0][0], r)[c.rank * kReqMaxRows + c.tid] = v;
  }
  cluster.sync();
}
__device__ __forceinline__ float req_norm_of(const ReqCtx& c, const ReqShared& S, int row) {
  unsigned long long t = 0;
  for (unsigned r = 0; r < c.CS; ++r) t += S.all_sum[r][row];
  return norm_of(t);
}

// This CTA's mass of one distribution (block sum), gathered into S.all_mass[which][rank] of every CTA.
// Ends with the cluster barrier.
__device__ __forceinline__ void req_gather_mass(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, unsigned long long mine, int which) {
  mine = warp_sum_u64(mine);
  if (c.lane == 0) S.scan[c.warp] = mine;
  __syncthreads();
  if (c.tid == 0) {
    unsigned long long t = 0;
#pragma unroll
    for (int w = 0; w < kReqWarps; ++w) t += S.scan[w];
    for (unsigned r = 0; r < c.CS; ++r) cluster.map_shared_rank(&S.all_mass[0][0], r)[which * kReqMaxCluster + c.rank] = t;
  }
  cluster.sync();
}

// Two block sums at once (buffers `which` and `which + 1`), one cluster barrier.
__device__ __forceinline__ void req_gather_mass2(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, unsigned long long m0,
                                                 unsigned long long m1, int which) {
  m0 = warp_sum_u64(m0); m1 = warp_sum_u64(m1);
  if (c.lane == 0) { S.scan[c.warp] = m0; S.scan2[c.warp] = m1; }
  __syncthreads();
  if (c.tid == 0) {
    unsigned long long t0 = 0, t1 = 0;
#pragma unroll
    for (int w = 0; w < kReqWarps; ++w) { t0 += S.scan[w]; t1 += S.scan2[w]; }
    for (unsigned r = 0; r < c.CS; ++r) {
      unsigned long long* dst = cluster.map_shared_rank(&S.all_mass[0][0], r);
      dst[which * kReqMaxCluster + c.rank] = t0;
      dst[(which + 1) * kReqMaxCluster + c.rank] = t1;
    }
  }
  cluster.sync();
}

// For the draw every thread owns a CONTIGUOUS range of the slice (so that a prefix over the threads is a prefix
// over the vocabulary): [t_lo, t_hi), a multiple of 4 elements long.
__device__ __forceinline__ void req_thread_range(const ReqCtx& c, int slice, int* t_lo, int* t_hi) {
  const int per = ((slice + kReqThreads - 1) / kReqThreads + 3) & ~3;
  *t_lo = min(c.v_hi, c.v_lo + c.tid * per);
  *t_hi = min(c.v_hi, *t_lo + per);
}

// Inverse-CDF draw on the masses gathered in S.all_mass[which] (tmass = this thread's mass over its range):
// the CTA whose slice holds the threshold finds the thread whose range holds it (one block-wide prefix sum),
// and that thread walks its range.  Returns true in every thread of that CTA only, with the token in *token.
// mass_at(v) gives the integer mass of element v.
template <typename MassAt>
__device__ __forceinline__ bool req_draw(const ReqCtx& c, ReqShared& S, int which, float u, unsigned long long tmass, int t_lo, int t_hi,
                                         MassAt mass_at, int* token, int* status) {
  unsigned long long T = 0;
  for (unsigned r = 0; r < c.CS; ++r) T += S.all_mass[which][r];
  *status = 0;
  if (T == 0ull) { *status = 1; return false; }               // no mass (caller decides: fall back or report)
  unsigned long long thr = draw_threshold(u, T);
  unsigned owner = 0;
  for (; owner + 1 < c.CS; ++owner) {
    const unsigned long long mr = S.all_mass[which][owner];
    if (thr < mr) break;
    thr -= mr;
  }
  if (owner != c.rank) return false;
  unsigned long long incl = tmass;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
    if (c.lane >= o) incl += t;
  }
  __syncthreads();                                             // (S.scan was read by the gather before)
  if (c.lane == 31) S.scan[c.warp] = incl;
  if (c.tid == 0) S.result = 0x7fffffff;
  __syncthreads();
  unsigned long long run = incl - tmass;
#pragma unroll
  for (int i = 0; i < kReqWarps; ++i) if (i < c.warp) run += S.scan[i];
  if (run <= thr && thr < run + tmass) {
#pragma unroll 1
    for (int v = t_lo; v < t_hi; ++v) {
      const unsigned long long mv = mass_at(v);
      run += mv;
      if (run > thr && mv != 0ull) { S.result = v; break; }
    }
  }
  __syncthreads();
  const int y = S.result;
  if (y == 0x7fffffff) { *status = 2; *token = 0; }           // cannot happen for consistent masses; reported
  else *token = y;
  return true;
}

__device__ __forceinline__ ReqCtx req_ctx(cg::cluster_group& cluster, int V, int slice) {
  ReqCtx c;
  c.CS = cluster.num_blocks(); c.rank = cluster.block_rank();
  c.tid = threadIdx.x; c.lane = c.tid & 31; c.warp = c.tid >> 5;
  c.v_lo = min(V, (int)c.rank * slice); c.v_hi = min(V, c.v_lo + slice);
  return c;
}

// per-thread best of a value over the slice -> block -> gathered over the cluster into S.all_best[r][row]
__device__ __forceinline__ void req_gather_best(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, ReqBest mine, int row, bool last_row) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    ReqBest other;
    other.val = __shfl_xor_sync(0xffffffffu, mine.val, o);
    other.idx = __shfl_xor_sync(0xffffffffu, mine.idx, o);
    best_merge(mine, other);
  }
  if (c.lane == 0) S.red_b[c.warp][row] = mine;
  if (!last_row) return;
  __syncthreads();
  if (c.tid <= row) {
    ReqBest v = S.red_b[0][c.tid];
#pragma unroll
    for (int w = 1; w < kReqWarps; ++w) best_merge(v, S.red_b[w][c.tid]);
    for (unsigned r = 0; r < c.CS; ++r) cluster.map_shared_rank(&S.all_best[0][0], r)[c.rank * kReqMaxRows + c.tid] = v;
  }
}
__device__ __forceinline__ int req_best_of(const ReqCtx& c, const ReqShared& S, int row) {
  ReqBest v = S.all_best[0][row];
  for (unsigned r = 1; r < c.CS; ++r) best_merge(v, S.all_best[r][row]);
  return v.idx;
}

// ------------------------------------------------------------------------------------------------
// Algorithm 1 steps 6-7 for one request per cluster.  logits [B][m][V] (row = b*m + k).
// ------------------------------------------------------------------------------------------------
struct EnsembleArgs {
  int V, m, greedy, slice;
  int D;                                        // candidates per step (1: a plain chain); candidate c uses u[.. + c]
  int* cand; int cand_stride;                   // optional: all candidates, cand[b * cand_stride + c] (-1: none left)
  const float* logits;
  const float* w;                               // [B][m]
  const float* u; int u_stride;                 // u[b * u_stride]
  float* qk_out; long long qk_req_stride;       // optional [b][k][V]
  float* q_out; long long q_req_stride;         // required (the draw re-reads it)
  int* out0; int out0_stride;                   // y[b * out0_stride]
  int* out1; int out1_stride;                   // optional second copy
  int* err;
  int ebuf_pitch;                               // > 0: the launch has m * ebuf_pitch floats of dynamic shared memory for the slices
};

extern __shared__ float4 req_dyn_smem[];

__global__ void __launch_bounds__(kReqThreads, 2) k_ensemble_req(const EnsembleArgs A) {
  pdl_trigger();
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ ReqShared S;
  const ReqCtx c = req_ctx(cluster, A.V, A.slice);
  const int b = blockIdx.x / c.CS, m = A.m, V = A.V;
  float* ebuf = A.ebuf_pitch > 0 ? reinterpret_cast<float*>(req_dyn_smem) : nullptr;
  const int epitch = A.ebuf_pitch;
  pdl_wait();
  const float* lg = A.logits + (long long)b * m * V;
  const bool vec = req_vec_ok(A.logits, V);
  req_row_maxima(cluster, c, S, lg, V, m, vec, ebuf, epitch);
  req_row_sums(cluster, c, S, lg, V, m, vec, ebuf, epitch);
  // (the loop over the inputs below is a real loop - the kernel's code runs once per CTA, so its size is what
  // the instruction fetch pays for - hence the rows' scalars sit in shared memory, not in registers)
  if (c.tid < m) {
    S.par[0][c.tid] = req_max_of(c, S, c.tid);
    S.par[1][c.tid] = req_norm_of(c, S, c.tid);
    S.par[2][c.tid] = A.w[b * m + c.tid];
  }
  __syncthreads();
  float* q_row = A.q_out + (long long)b * A.q_req_stride;
  float* qk_b = A.qk_out ? A.qk_out + (long long)b * A.qk_req_stride : nullptr;
  const bool vec_q = req_vec_ok(A.q_out, A.q_req_stride) && (V & 3) == 0;
  const bool vec_qk = A.qk_out && req_vec_ok(A.qk_out, A.qk_req_stride) && (V & 3) == 0;
  unsigned long long mass = 0;
  ReqBest best{-1.0f, 0x7fffffff};
#pragma unroll 1
  for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
    float acc[4];
    float nxt[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (!ebuf) req_ld4(lg, v, c.v_hi, vec, -INFINITY, nxt);
#pragma unroll 1
    for (int k = 0; k < m; ++k) {
      float a[4];
      const float mxk = S.par[0][k], snk = S.par[1][k], wkk = S.par[2][k];
      if (ebuf) {
        const float4 t = *reinterpret_cast<const float4*>(ebuf + (size_t)k * epitch + (v - c.v_lo));     // the exponentials
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) a[j] = xexp(__fsub_rn(nxt[j], mxk));
        if (k + 1 < m) req_ld4(lg + (long long)(k + 1) * V, v, c.v_hi, vec, -INFINITY, nxt);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        a[j] = __fdiv_rn(a[j], snk);
        const float t = __fmul_rn(wkk, a[j]);
        acc[j] = (k == 0) ? t : __fadd_rn(acc[j], t);
      }
      if (qk_b) req_st4(qk_b + (long long)k * V, v, c.v_hi, vec_qk, a);
    }
    req_st4(q_row, v, c.v_hi, vec_q, acc);
    if (A.greedy) {
#pragma unroll
      for (int j = 0; j < 4; ++j) if (v + j < c.v_hi && acc[j] > best.val) { best.val = acc[j]; best.idx = v + j; }
    }
  }
  // the step's candidates: candidate 0 continues the chain; further ones (token tree) are drawn without replacement
  const int D = A.D;
  int chosen[kReqMaxWidth] = {-1, -1, -1, -1};
  auto emit = [&](int cnd, int y) {
    if (cnd == 0) A.out0[b * A.out0_stride] = y;
    if (A.out1) A.out1[b * A.out1_stride + cnd] = y;
    if (A.cand) A.cand[b * A.cand_stride + cnd] = y;
  };
  if (A.greedy) {
#pragma unroll 1
    for (int cnd = 0; cnd < D; ++cnd) {
      if (cnd > 0) {
        // most likely token among those not chosen yet (the slice was written by this CTA: L1/L2 hold it)
        best = ReqBest{-1.0f, 0x7fffffff};
        __syncthreads();
#pragma unroll 1
        for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
          float x[4];
          req_ld4_rw(q_row, v, c.v_hi, vec_q, -1.0f, x);
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int t = v + j;
            if (t < c.v_hi && t != chosen[0] && t != chosen[1] && t != chosen[2] && x[j] > best.val) { best.val = x[j]; best.idx = t; }
          }
        }
      }
      // (the merge of the warps' bests uses one row of the exchange buffers per candidate)
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ReqBest other;
        other.val = __shfl_xor_sync(0xffffffffu, best.val, o);
        other.idx = __shfl_xor_sync(0xffffffffu, best.idx, o);
        best_merge(best, other);
      }
      if (c.lane == 0) S.red_b[c.warp][cnd] = best;
      __syncthreads();
      if (c.tid == 0) {
        ReqBest t = S.red_b[0][cnd];
#pragma unroll
        for (int w = 1; w < kReqWarps; ++w) best_merge(t, S.red_b[w][cnd]);
        for (unsigned r = 0; r < c.CS; ++r) cluster.map_shared_rank(&S.all_best[0][0], r)[c.rank * kReqMaxRows + cnd] = t;
      }
      cluster.sync();
      ReqBest t = S.all_best[0][cnd];
      for (unsigned r = 1; r < c.CS; ++r) best_merge(t, S.all_best[r][cnd]);
      const int y = t.val < 0.0f ? -1 : t.idx;              // fewer tokens than candidates
      chosen[cnd] = y;
      if (c.rank == 0 && c.tid == 0) emit(cnd, y);
    }
    return;
  }
  // masses of q over each thread's contiguous range (the slice was just written by this CTA: L1/L2 hold it)
  __syncthreads();
  int t_lo, t_hi;
  req_thread_range(c, A.slice, &t_lo, &t_hi);
#pragma unroll 1
  for (int v = t_lo; v < t_hi; v += 4) {
    float x[4];
    req_ld4_rw(q_row, v, t_hi, vec_q, 0.0f, x);
#pragma unroll
    for (int j = 0; j < 4; ++j) if (v + j < t_hi) mass += mass_of(x[j]);
  }
  req_gather_mass(cluster, c, S, mass, 0);
  auto mass_left = [&](int v) { return (v == chosen[0] || v == chosen[1] || v == chosen[2]) ? 0ull : mass_of(q_row[v]); };
#pragma unroll 1
  for (int cnd = 0; cnd < D; ++cnd) {
    int y = 0, status = 0;
    const bool mine = req_draw(c, S, 0, A.u[b * A.u_stride + cnd], mass, t_lo, t_hi, mass_left, &y, &status);
    if (status == 1) {
      // nothing (left) to draw from: an error for the chain's own token, "no candidate" for a sibling
      if (c.rank == 0 && c.tid == 0) {
        if (cnd == 0) { if (A.err) atomicOr(A.err, 1); emit(0, 0); }
        for (int k = cnd > 0 ? cnd : 1; k < D; ++k) emit(k, -1);
      }
      break;
    }
    if (mine && c.tid == 0) {
      if (status && A.err) atomicOr(A.err, status);
      emit(cnd, y);
    }
    if (cnd + 1 == D) break;
    // tell every CTA which token went and how much mass leaves with it
    if (mine && c.tid == 0) {
      const unsigned long long my = (status == 0) ? mass_of(q_row[y]) : 0ull;
      for (unsigned r = 0; r < c.CS; ++r) {
        cluster.map_shared_rank(&S.bc_tok[0], r)[cnd] = (status == 0) ? y : -1;
        cluster.map_shared_rank(&S.bc_mass[0], r)[cnd] = my;
      }
    }
    cluster.sync();
    const int yt = S.bc_tok[cnd];
    chosen[cnd] = yt;
    if (yt >= 0) {
      const unsigned long long my = S.bc_mass[cnd];
      if (c.tid == 0) S.all_mass[0][yt / A.slice] -= my;
      if (yt >= t_lo && yt < t_hi) mass -= my;
      __syncthreads();
    }
  }
}

// A cluster reports that its part of request b is in global memory and learns whether it is the last of
// `n_parts`: the block barrier (the caller's cluster barrier) orders the cluster's stores before the fence of
// CTA 0's first thread, which takes the ticket; the last arriver resets it.  Ends with a cluster barrier; the
// answer is the same in every thread of the cluster.
__device__ __forceinline__ bool req_last_of_request(cg::cluster_group& cluster, const ReqCtx& c, int* flag_smem, int* ticket, int n_parts) {
  if (c.rank == 0 && c.tid == 0) {
    __threadfence();
    const int last = atomicAdd(ticket, 1) == n_parts - 1;
    if (last) { *ticket = 0; __threadfence(); }
    for (unsigned r = 0; r < c.CS; ++r) *cluster.map_shared_rank(flag_smem, r) = last;
  }
  cluster.sync();
  return *flag_smem != 0;
}

// ------------------------------------------------------------------------------------------------
// Sec. 3 item 3.  grid: B * (G + 1) clusters; cluster (b, i) owns target row i of request b.
// ------------------------------------------------------------------------------------------------
struct VerifyArgs {
  int V, G, greedy, slice;
  int D;                                        // candidates per depth (token tree; 1: a plain chain)
  const float* logits;                          // target [B][Rt][V], Rt = G + 1 + G (D - 1): the chain's positions, then the
                                                // leaf after sibling c of depth i at row G + 1 + i (D - 1) + (c - 1)
  const float* q; long long q_req_stride;       // ensembled [B][..][V], position pitch V
  const int* tokens;                            // [B][G] the primary chain
  const int* cand;                              // [B][G][D] all candidates (column 0 = tokens)
  const float* u_accept;                        // [B][G][D]
  const float* u_resid;                         // [B]
  float* p;                                     // [B][Rt][V]
  int *acc_prim, *sib_tok;                      // [B] accepted tokens of the primary chain; the accepted sibling's token or -1
  int* row_flag;                                // [B][G+1] scratch: accept flag of position i (greedy: argmax of p_i)
  int* ticket;                                  // [B] scratch, zero between launches
  int *n_accept, *out_n_accept, *next_token, *out_next_token;
  int* err;
  int ebuf_pitch;                               // > 0: the launch has ebuf_pitch floats of dynamic shared memory for the row's slice
  int tail_inline;                              // 1: the request's last cluster runs the tail; 0: k_verify_tail does (a launch of
                                                // its own with one LARGE cluster per request - with many requests the clusters
                                                // of this kernel are small and the tail would crawl through a row on 1-2 CTAs)
};

__device__ __forceinline__ void verify_tail(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, const VerifyArgs& A, int b);

__global__ void __launch_bounds__(kReqThreads, 2) k_verify_req(const VerifyArgs A) {
  pdl_trigger();
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ ReqShared S;
  __shared__ int s_last;
  const ReqCtx c = req_ctx(cluster, A.V, A.slice);
  const int G = A.G, V = A.V, rows = G + 1, D = A.D, Rt = G + 1 + G * (D - 1);
  const int unit = blockIdx.x / c.CS, b = unit / rows, i = unit - b * rows;
  pdl_wait();
  const float* lg = A.logits + ((long long)b * Rt + i) * V;
  float* p_b = A.p + (long long)b * Rt * V;
  const float* q_b = A.q + (long long)b * A.q_req_stride;
  const bool vec = req_vec_ok(A.logits, V), vec_p = (V & 3) == 0;
  float* ebuf = A.ebuf_pitch > 0 ? reinterpret_cast<float*>(req_dyn_smem) : nullptr;
  req_row_maxima(cluster, c, S, lg, V, 1, vec, ebuf, A.ebuf_pitch);
  req_row_sums(cluster, c, S, lg, V, 1, vec, ebuf, A.ebuf_pitch);
  const float mx = req_max_of(c, S, 0), sn = req_norm_of(c, S, 0);
  {
    // p_i = e / S; in greedy mode also its argmax
    ReqBest best{-1.0f, 0x7fffffff};
#pragma unroll 1
    for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
      float a[4];
      if (ebuf) {
        const float4 t = *reinterpret_cast<const float4*>(ebuf + (v - c.v_lo));                       // the exponentials
        a[0] = t.x; a[1] = t.y; a[2] = t.z; a[3] = t.w;
      } else {
        req_ld4(lg, v, c.v_hi, vec, -INFINITY, a);
#pragma unroll
        for (int j = 0; j < 4; ++j) a[j] = xexp(__fsub_rn(a[j], mx));
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        a[j] = __fdiv_rn(a[j], sn);
        if (A.greedy && v + j < c.v_hi && a[j] > best.val) { best.val = a[j]; best.idx = v + j; }
      }
      req_st4(p_b + (long long)i * V, v, c.v_hi, vec_p, a);
    }
    if (A.greedy) req_gather_best(cluster, c, S, best, 0, true);
  }
  cluster.sync();                                // the row is stored (and the bests gathered)
  if (c.rank == 0 && c.tid == 0) {
    int flag;
    if (A.greedy) flag = req_best_of(c, S, 0);
    else if (i < G) {
      const int y = A.tokens[b * G + i];
      const float py = __fdiv_rn(xexp(__fsub_rn(__ldg(lg + y), mx)), sn);          // the value stored in p_i[y]
      const float qy = __ldg(q_b + (long long)i * V + y);
      flag = (py >= qy) || (__fmul_rn(A.u_accept[(b * G + i) * D], qy) < py);
    } else flag = 1;
    A.row_flag[b * rows + i] = flag;
  }
  if (!A.tail_inline) return;
  if (!req_last_of_request(cluster, c, &s_last, A.ticket + b, rows)) return;
  verify_tail(cluster, c, S, A, b);
}

// The tail alone: one cluster per request, after k_verify_req (tail_inline = 0) has stored p and the row flags.
__global__ void __launch_bounds__(kReqThreads, 2) k_verify_tail(const VerifyArgs A) {
  pdl_trigger();
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ ReqShared S;
  const ReqCtx c = req_ctx(cluster, A.V, A.slice);
  pdl_wait();
  verify_tail(cluster, c, S, A, (int)(blockIdx.x / c.CS));
}

// ---- per request: acceptance prefix, siblings of the first rejected depth, next token (Sec. 3 item 3; Sec. 5 token tree) ----
__device__ __forceinline__ void verify_tail(cg::cluster_group& cluster, const ReqCtx& c, ReqShared& S, const VerifyArgs& A, int b) {
  const int G = A.G, V = A.V, rows = G + 1, D = A.D, Rt = G + 1 + G * (D - 1);
  float* p_b = A.p + (long long)b * Rt * V;
  const float* q_b = A.q + (long long)b * A.q_req_stride;
  const bool vec = req_vec_ok(A.logits, V), vec_p = (V & 3) == 0;
  int a = 0;
  for (; a < G; ++a) {
    const int f = __ldcg(A.row_flag + b * rows + a);
    if (A.greedy ? (f != A.tokens[b * G + a]) : (f == 0)) break;
  }
  const float u = A.u_resid[b];
  int t_lo, t_hi;
  req_thread_range(c, A.slice, &t_lo, &t_hi);
  int n_acc = a, sib = -1, z = 0, status = 0;
  bool mine = false, have_z = false;
  // Next token from the target's distribution of one row, computed here (a leaf of the tree): softmax, then draw / argmax.
  auto from_row = [&](int row) {
    const float* lr = A.logits + ((long long)b * Rt + row) * V;
    float* pr = p_b + (long long)row * V;
    req_row_maxima(cluster, c, S, lr, V, 1, vec);
    req_row_sums(cluster, c, S, lr, V, 1, vec);
    const float mx2 = req_max_of(c, S, 0), sn2 = req_norm_of(c, S, 0);
    unsigned long long mass = 0;
    ReqBest best{-1.0f, 0x7fffffff};
#pragma unroll 1
    for (int v = t_lo; v < t_hi; v += 4) {
      float x[4];
      req_ld4(lr, v, t_hi, vec, -INFINITY, x);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        x[j] = __fdiv_rn(xexp(__fsub_rn(x[j], mx2)), sn2);
        if (v + j < t_hi) { mass += mass_of(x[j]); if (x[j] > best.val) { best.val = x[j]; best.idx = v + j; } }
      }
      req_st4(pr, v, t_hi, vec_p, x);
    }
    if (A.greedy) {
      req_gather_best(cluster, c, S, best, 0, true);
      cluster.sync();
      z = req_best_of(c, S, 0);
      mine = c.rank == 0;
    } else {
      req_gather_mass(cluster, c, S, mass, 0);
      mine = req_draw(c, S, 0, u, mass, t_lo, t_hi,
                      [&](int v) { return mass_of(__fdiv_rn(xexp(__fsub_rn(__ldg(lr + v), mx2)), sn2)); }, &z, &status);
      if (status == 1 && c.rank == 0) { mine = true; z = 0; }
    }
  };
  if (A.greedy) {
    if (a < G) {
      const int t = __ldcg(A.row_flag + b * rows + a);            // the target's token at the first depth that differs
      for (int cnd = 1; cnd < D; ++cnd) if (sib < 0 && A.cand[(b * G + a) * D + cnd] == t) sib = cnd;
      if (sib < 0) { z = t; mine = c.rank == 0; have_z = true; }
    } else {
      z = __ldcg(A.row_flag + b * rows + G); mine = c.rank == 0; have_z = true;
    }
  } else if (a < G) {
    // Recursive rejection over the depth's candidates.  Level l distributions are functions of (p_a, q_a) and of the
    // scalars of the levels before: r = max(0, p - q); p' = r / Rn; q' = q / Qn with the tried tokens at 0.
    const float* p_a = p_b + (long long)a * V;                   // written by another cluster of this launch: read through L2
    const float* q_a = q_b + (long long)a * V;
    float Rn[kReqMaxWidth], Qn[kReqMaxWidth];
    int xs[kReqMaxWidth];
#pragma unroll
    for (int k = 0; k < kReqMaxWidth; ++k) { xs[k] = k < D ? A.cand[(b * G + a) * D + k] : -1; Rn[k] = 1.0f; Qn[k] = 1.0f; }
    auto elem = [&](int v, int level, float& pl, float& ql) {
      pl = __ldcg(p_a + v); ql = __ldg(q_a + v);
#pragma unroll
      for (int l = 1; l < kReqMaxWidth; ++l) {
        if (l > level) break;
        const float r = resid_val(pl, ql);
        pl = __fdiv_rn(r, Rn[l]);
        ql = (v == xs[l - 1]) ? 0.0f : __fdiv_rn(ql, Qn[l]);
      }
    };
    int level = 0;
#pragma unroll 1
    while (true) {
      // this level's residual masses (per thread range) and the mass of q_level
      unsigned long long mr = 0, mq = 0;
#pragma unroll 1
      for (int v = t_lo; v < t_hi; ++v) {
        float pl, ql;
        elem(v, level, pl, ql);
        mr += mass_of(resid_val(pl, ql));
        mq += mass_of(ql);
      }
      const int buf = 2 * (level & 1);
      req_gather_mass2(cluster, c, S, mr, mq, buf);
      unsigned long long MR = 0, MQ = 0;
      for (unsigned r = 0; r < c.CS; ++r) { MR += S.all_mass[buf][r]; MQ += S.all_mass[buf + 1][r]; }
      float px, qx;
      elem(xs[level], level, px, qx);
      const unsigned long long MQrest = MQ - mass_of(qx);
      const bool more = level + 1 < D && xs[level + 1] >= 0 && MR != 0ull && MQrest != 0ull;
      if (!more) {
        // the replacement: from this level's residual, or from p_level itself if that has no mass
        if (MR != 0ull) {
          mine = req_draw(c, S, buf, u, mr, t_lo, t_hi,
                          [&](int v) { float pl, ql; elem(v, level, pl, ql); return mass_of(resid_val(pl, ql)); }, &z, &status);
        } else {
          unsigned long long mp = 0;
#pragma unroll 1
          for (int v = t_lo; v < t_hi; ++v) { float pl, ql; elem(v, level, pl, ql); mp += mass_of(pl); }
          req_gather_mass(cluster, c, S, mp, buf ^ 2);
          mine = req_draw(c, S, buf ^ 2, u, mp, t_lo, t_hi, [&](int v) { float pl, ql; elem(v, level, pl, ql); return mass_of(pl); }, &z, &status);
        }
        if (status == 1 && c.rank == 0) { mine = true; z = 0; }
        have_z = true;
        break;
      }
      Rn[level + 1] = norm_of(MR);
      Qn[level + 1] = norm_of(MQrest);
      ++level;
      elem(xs[level], level, px, qx);
      if ((px >= qx) || (__fmul_rn(A.u_accept[(b * G + a) * D + level], qx) < px)) { sib = level; break; }
    }
  }
  if (sib >= 0) {
    n_acc = a + 1;
    from_row(G + 1 + a * (D - 1) + (sib - 1));                   // the leaf after the accepted sibling
  } else if (!have_z) {
    // every primary accepted: bonus token from p_G
    const float* p_g = p_b + (long long)G * V;
    unsigned long long mass = 0;
#pragma unroll 1
    for (int v = t_lo; v < t_hi; v += 4) {
      float x[4];
      if (vec_p && v + 4 <= t_hi) { const float4 t = __ldcg(reinterpret_cast<const float4*>(p_g + v)); x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w; }
      else { for (int j = 0; j < 4; ++j) x[j] = (v + j < t_hi) ? __ldcg(p_g + v + j) : 0.0f; }
#pragma unroll
      for (int j = 0; j < 4; ++j) if (v + j < t_hi) mass += mass_of(x[j]);
    }
    req_gather_mass(cluster, c, S, mass, 0);
    mine = req_draw(c, S, 0, u, mass, t_lo, t_hi, [&](int v) { return mass_of(__ldcg(p_g + v)); }, &z, &status);
    if (status == 1 && c.rank == 0) { mine = true; z = 0; }
  }
  if (c.rank == 0 && c.tid == 0) {
    A.n_accept[b] = n_acc;
    if (A.out_n_accept) A.out_n_accept[b] = n_acc;
    A.acc_prim[b] = a;
    A.sib_tok[b] = sib >= 0 ? A.cand[(b * G + a) * D + sib] : -1;
  }
  if (mine && c.tid == 0) {
    if (status && A.err) atomicOr(A.err, status);
    A.next_token[b] = z;
    if (A.out_next_token) A.out_next_token[b] = z;
  }
}

// ------------------------------------------------------------------------------------------------
// Sec. 4.1 / App. B.  grid: B * G clusters; cluster (b, i) sums the deviations of position i (if it is a
// verified one: i <= min(a, G-1)); the fixed-point partial sums of its CTAs meet in CTA 0 (integer sums:
// order-free), which stores them; the last cluster of the request then runs the policy in one warp.
// ------------------------------------------------------------------------------------------------
struct UpdateArgs {
  int V, slice, grid_policy;
  int Rt;                         // rows of p per request (G + 1, more with a token tree)
  int hard;                       // 0: soft labels (distance sums); 1: hard labels - whether each grid candidate's most likely
                                  // token is the verified token (matches); 2: whether each drafter's is NOT (errors)
  const float* p;                 // [B][Rt][V]
  const float* qk;                // [B][G][m][V]
  int* ticket;                    // [B] scratch, zero between launches
  PolicyArgs P;                   // P.dev: [B][G][kMaxDev] scratch (every verified entry is rewritten each round)
};

struct UpdShared {
  long long red[kReqWarps][kMaxDev];
  long long all_dev[kReqMaxCluster][kMaxDev];        // [CTA][deviation index], filled in CTA 0
  ReqBest red_b[kReqWarps][kMaxDev];                 // hard labels: most likely token per candidate
  ReqBest all_b[kReqMaxCluster][kMaxDev];
};

__device__ __forceinline__ void policy_commit(const PolicyArgs& A, int b, int lane, int last);

__global__ void __launch_bounds__(kReqThreads, 2) k_update_req(const UpdateArgs A) {
  pdl_trigger();
  cg::cluster_group cluster = cg::this_cluster();
  __shared__ UpdShared U;
  __shared__ int s_last;
  const ReqCtx c = req_ctx(cluster, A.V, A.slice);
  const PolicyArgs& P = A.P;
  const int G = P.G, V = A.V, m = P.m, n_dev = P.n_dev, tvd = P.tvd;
  const int unit = blockIdx.x / c.CS, b = unit / G, i = unit - b * G;
  pdl_wait();
  const int a = P.n_accept[b];
  const int last = min(a, G - 1);
  if (i > last) return;                             // (the whole cluster: position not verified)
  const bool vec = (V & 3) == 0;
  // The loops over the deviation index (drafter or grid candidate) are real loops with the accumulators in local
  // memory: the kernel's code runs once per CTA, so its size is what the instruction fetch pays for.
  const float* qbase = A.qk + ((long long)b * G + i) * m * V;
  if (A.hard) {
    // most likely token (lowest id on ties) of every grid candidate's ensemble, or of every drafter
    ReqBest best[kMaxDev];
#pragma unroll 1
    for (int kd = 0; kd < n_dev; ++kd) best[kd] = ReqBest{-1.0f, 0x7fffffff};
#pragma unroll 1
    for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
      float q0[4], q1[4];
      if (A.grid_policy) {
        req_ld4(qbase, v, c.v_hi, vec, 0.0f, q0);
        req_ld4(qbase + V, v, c.v_hi, vec, 0.0f, q1);
      }
#pragma unroll 1
      for (int kd = 0; kd < n_dev; ++kd) {
        float x[4];
        if (A.grid_policy) {
          const float c1 = __fdiv_rn((float)kd, 10.0f);
          const float c0 = __fsub_rn(1.0f, c1);
#pragma unroll
          for (int j = 0; j < 4; ++j) x[j] = __fadd_rn(__fmul_rn(c0, q0[j]), __fmul_rn(c1, q1[j]));
        } else {
          req_ld4(qbase + (long long)kd * V, v, c.v_hi, vec, 0.0f, x);
        }
        ReqBest t = best[kd];
#pragma unroll
        for (int j = 0; j < 4; ++j) if (v + j < c.v_hi && x[j] > t.val) { t.val = x[j]; t.idx = v + j; }
        best[kd] = t;
      }
    }
#pragma unroll 1
    for (int kd = 0; kd < n_dev; ++kd) {
      ReqBest mine = best[kd];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ReqBest other;
        other.val = __shfl_xor_sync(0xffffffffu, mine.val, o);
        other.idx = __shfl_xor_sync(0xffffffffu, mine.idx, o);
        best_merge(mine, other);
      }
      if (c.lane == 0) U.red_b[c.warp][kd] = mine;
    }
    __syncthreads();
    if (c.tid < n_dev) {
      ReqBest t = U.red_b[0][c.tid];
#pragma unroll 1
      for (int w = 1; w < kReqWarps; ++w) best_merge(t, U.red_b[w][c.tid]);
      cluster.map_shared_rank(&U.all_b[0][0], 0)[c.rank * kMaxDev + c.tid] = t;
    }
    cluster.sync();
    if (c.rank == 0 && c.tid < n_dev) {
      ReqBest t = U.all_b[0][c.tid];
      for (unsigned r = 1; r < c.CS; ++r) best_merge(t, U.all_b[r][c.tid]);
      // the verified token of position i: the accepted draft, or the replacement at the rejected position
      const int sib = P.sib_tok[b];
      const int label = (i < a) ? P.tokens[b * G + i] : (sib >= 0 ? sib : P.next_token[b]);
      const int hit = t.idx == label;
      P.dev[((long long)b * G + i) * kMaxDev + c.tid] = (A.hard == 1) ? hit : 1 - hit;
    }
  } else {
    const float* p_i = A.p + ((long long)b * A.Rt + i) * V;
    long long acc[kMaxDev];
#pragma unroll 1
    for (int kd = 0; kd < n_dev; ++kd) acc[kd] = 0;
#pragma unroll 1
    for (int v = c.v_lo + c.tid * 4; v < c.v_hi; v += kReqStep) {
      float pv[4], lp[4], q0[4], q1[4], nxt[4];
      req_ld4(p_i, v, c.v_hi, vec, 0.0f, pv);
      if (A.grid_policy) {
        req_ld4(qbase, v, c.v_hi, vec, 0.0f, q0);
        req_ld4(qbase + V, v, c.v_hi, vec, 0.0f, q1);
      } else {
        req_ld4(qbase, v, c.v_hi, vec, 0.0f, nxt);
      }
      if (!tvd) {
#pragma unroll
        for (int j = 0; j < 4; ++j) lp[j] = xlog(fmaxf(pv[j], kFltMin));
      }
#pragma unroll 1
      for (int kd = 0; kd < n_dev; ++kd) {
        float x[4];
        if (A.grid_policy) {
          const float c1 = __fdiv_rn((float)kd, 10.0f);
          const float c0 = __fsub_rn(1.0f, c1);
#pragma unroll
          for (int j = 0; j < 4; ++j) x[j] = __fadd_rn(__fmul_rn(c0, q0[j]), __fmul_rn(c1, q1[j]));
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j) x[j] = nxt[j];
          if (kd + 1 < n_dev) req_ld4(qbase + (long long)(kd + 1) * V, v, c.v_hi, vec, 0.0f, nxt);      // the next row while this one is worked on
        }
        long long sum = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (v + j >= c.v_hi) continue;
          float t;
          if (tvd) t = fabsf(__fsub_rn(pv[j], x[j]));
          else t = (pv[j] > 0.0f) ? __fmul_rn(pv[j], __fsub_rn(lp[j], xlog(fmaxf(x[j], kFltMin)))) : 0.0f;
          sum += __float2ll_rz(__fmul_rn(t, kMassScale));
        }
        acc[kd] += sum;
      }
    }
#pragma unroll 1
    for (int kd = 0; kd < n_dev; ++kd) {
      const long long t = warp_sum_i64(acc[kd]);
      if (c.lane == 0) U.red[c.warp][kd] = t;
    }
    __syncthreads();
    if (c.tid < n_dev) {
      long long t = 0;
#pragma unroll 1
      for (int w = 0; w < kReqWarps; ++w) t += U.red[w][c.tid];
      cluster.map_shared_rank(&U.all_dev[0][0], 0)[c.rank * kMaxDev + c.tid] = t;
    }
    cluster.sync();
    if (c.rank == 0 && c.tid < n_dev) {
      long long t = 0;
      for (unsigned r = 0; r < c.CS; ++r) t += U.all_dev[r][c.tid];
      P.dev[((long long)b * G + i) * kMaxDev + c.tid] = t;
    }
  }
  __syncthreads();                                  // (CTA 0: the sums are stored before its first thread's fence)
  if (!req_last_of_request(cluster, c, &s_last, A.ticket + b, last + 1)) return;
  if (c.rank == 0 && c.warp == 0) policy_commit(P, b, c.lane, last);
}

// One warp per request: lane kd carries deviation index kd through the window (its running sum stays in a
// register), then lane 0 applies the policy in its fixed order and commits the caches and pending tokens.
__device__ __forceinline__ void policy_commit(const PolicyArgs& A, int b, int lane, int last) {
  const int a = A.n_accept[b];
  long long r = 0;
  {
    long long* run = A.running + (long long)b * kMaxDev;
    const bool on = lane < A.n_dev;
    if (on) r = run[lane];
    int head = A.h > 0 ? A.ring_head[b] : 0, count = A.h > 0 ? A.ring_count[b] : 0;
    for (int i = 0; i <= last; ++i) {
      const long long dv = on ? __ldcg(A.dev + ((long long)b * A.G + i) * kMaxDev + lane) : 0;   // stored by this launch's clusters
      if (A.h > 0) {
        long long* slot = A.ring + ((long long)b * A.h + head) * kMaxDev;
        const bool full = count == A.h;
        if (on) {
          if (full) r -= slot[lane];
          slot[lane] = dv;
        }
        head = (head + 1) % A.h;
        if (!full) count += 1;
      }
      r += dv;
    }
    if (on) run[lane] = r;
    if (lane == 0) {
      if (A.h > 0) { A.ring_head[b] = head; A.ring_count[b] = count; }
      A.pushed[b] += last + 1;
    }
  }
  long long run[kMaxDev];
#pragma unroll
  for (int kd = 0; kd < kMaxDev; ++kd) run[kd] = __shfl_sync(0xffffffffu, r, kd);
  if (lane != 0) return;
  const long long pushed = A.pushed[b];

  float* w = A.w + (long long)b * A.m;
  const float fx_scale = A.tvd ? 4.547473508864641e-13f : kMassInv;     // 2^-41 or 2^-40
  if (A.policy == 3) {
    // random point of the simplex from the caller's uniforms: g_k = -ln u_k, w_k = g_k / sum g
    float g[8], tot = 0.0f;
    for (int k = 0; k < A.m; ++k) {
      g[k] = -xlog(A.u_policy[(long long)b * A.m + k]);
      tot = (k == 0) ? g[0] : __fadd_rn(tot, g[k]);
    }
    for (int k = 0; k < A.m; ++k) w[k] = __fdiv_rn(g[k], tot);
  } else if (A.policy == 0 || pushed == 0) {
    const float s = __fdiv_rn(1.0f, (float)A.m);
    for (int k = 0; k < A.m; ++k) w[k] = s;
  } else if (A.policy == 5) {
    // AdaBoost-style weights from the drafters' error counts over the n window positions
    const long long n = A.h > 0 ? (long long)A.ring_count[b] : pushed;
    const float den = __fadd_rn(__ll2float_rn(n), 2.0f);
    const float lk = __fmul_rn(A.tau, xlog((float)(A.V - 1)));
    float t[8], tot = 0.0f;
    for (int k = 0; k < A.m; ++k) {
      const float eps = __fdiv_rn(__fadd_rn(__ll2float_rn(run[k]), 1.0f), den);
      t[k] = fmaxf(__fadd_rn(xlog(__fsub_rn(__fdiv_rn(1.0f, eps), 1.0f)), lk), 0.0f);
      tot = (k == 0) ? t[0] : __fadd_rn(tot, t[k]);
    }
    if (tot > 0.0f) { for (int k = 0; k < A.m; ++k) w[k] = __fdiv_rn(t[k], tot); }
    else { const float s = __fdiv_rn(1.0f, (float)A.m); for (int k = 0; k < A.m; ++k) w[k] = s; }
  } else if (A.policy == 1 || A.policy == 4) {
    // grid: least accumulated distance (soft labels) or most token matches (hard labels), lowest j on ties
    int js = 0;
    if (A.policy == 1) { for (int j = 1; j < kGridCand; ++j) if (run[j] < run[js]) js = j; }
    else { for (int j = 1; j < kGridCand; ++j) if (run[j] > run[js]) js = j; }
    A.grid_j[b] = js;
    const float c1 = __fdiv_rn((float)js, 10.0f);
    w[0] = __fsub_rn(1.0f, c1);
    w[1] = c1;
  } else {
    float s[8], x[8];
    float smax = -INFINITY;
    for (int k = 0; k < A.m; ++k) {
      const float e = __fmul_rn(__ll2float_rn(run[k]), fx_scale);
      s[k] = __fdiv_rn(1.0f, fmaxf(e, __uint_as_float(0x322BCC77u)));   // 1e-8
      smax = fmaxf(smax, s[k]);
    }
    float tot = 0.0f;
    for (int k = 0; k < A.m; ++k) {
      x[k] = xexp(__fdiv_rn(__fsub_rn(s[k], smax), A.tau));
      tot = (k == 0) ? x[0] : __fadd_rn(tot, x[k]);
    }
    for (int k = 0; k < A.m; ++k) w[k] = __fdiv_rn(x[k], tot);
  }
  int am = 0;
  for (int k = 1; k < A.m; ++k) if (w[k] > w[am]) am = k;
  if (A.out_w) for (int k = 0; k < A.m; ++k) A.out_w[(long long)b * A.m + k] = w[k];
  if (A.out_argmax) A.out_argmax[b] = am;

  // commit: caches keep the pending token(s) and the accepted drafts that were fed
  int* pend = A.pending + b * 3;
  const int cnt = pend[0];
  if (A.kv_len) {
    const int keep = cnt + (a < A.G ? a : A.G - 1);
    for (int k = 0; k < A.m; ++k) A.kv_len[b * A.m + k] += keep;
  }
  // ... and what the target emitted beyond them is pending: the replacement; or an accepted sibling (token tree) or the
  // last accepted draft of a fully accepted block, followed by the next token
  const int z = A.next_token[b], sib = A.sib_tok[b];
  if (a == A.G) { pend[0] = 2; pend[1] = A.tokens[b * A.G + A.G - 1]; pend[2] = z; }
  else if (sib >= 0) { pend[0] = 2; pend[1] = sib; pend[2] = z; }
  else { pend[0] = 1; pend[1] = z; pend[2] = 0; }
}

}  // namespace tabed
