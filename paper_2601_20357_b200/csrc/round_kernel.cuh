// Persistent kernel for one whole drafting round (Algorithm 1 steps 4-8): gamma batched
// shared-weight decoder steps, each followed by softmax + weighted-average ensemble + draw, in ONE
// cooperative launch with one CTA per SM.
//
// Why one kernel: with m <= 4 drafting inputs a decoder step moves ~125-630 MB of weights through
// ~25-65 strictly dependent phases; as separate launches every phase pays a launch plus a cold
// DRAM round trip.  Here
//   * the weights never stop streaming: every CTA owns a fixed, round-robin share of the weight
//     tiles of every phase, and one warp keeps a ring of shared-memory slots filled with bulk
//     asynchronous copies (cp.async.bulk + mbarrier) several phases ahead of the arithmetic, so
//     HBM stays busy across the grid barriers;
//   * a phase is: grid barrier -> stage the (tiny) activations from L2 -> tensor-core products
//     of the 16-row weight tiles already sitting in shared memory -> results back to L2;
//   * projections use mma.sync m16n8k16 (bf16 x bf16 -> fp32): 16 weight rows x up to 8 slots.
//     The contraction is HBM-bound (<= 8 flop per weight byte), the tensor pipe is used only to
//     keep the ALUs off the critical path;
//   * all cross-CTA data is read with ld.global.cg (L2) because L1 is not coherent across SMs.
//
// Waits are bounded: a grid barrier or a copy that does not complete within the spin limit sets an
// error bit, the CTA drains its copies in flight and returns.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "decide_kernels.cuh"
#include "exact_math.cuh"
#include "forward_kernels.cuh"

namespace tabed {

constexpr int kPT = 512;                 // threads per CTA
constexpr int kPW = kPT / 32;            // warps per CTA
constexpr int kPSlots = 8;               // slots (row, position) per step: one mma n-tile
constexpr int kPRing = 16;               // upper bound of ring slots
constexpr int kPPer = kChunk / kPT;      // vocabulary elements per thread and chunk (4)
constexpr int kPMaxD = 2048;             // d_model bound (4 residual elements per thread and slot)
constexpr int kPXE = kPMaxD / kPT;

enum { KIND_QKV = 0, KIND_O = 1, KIND_GU = 2, KIND_DN = 3, KIND_LM = 4 };
enum { PERR_BARRIER = 8, PERR_COPY = 16, PERR_KV = 4 };

struct LayerW { const __nv_bfloat16 *wq, *wk, *wv, *wo, *wg, *wu, *wd, *n1, *n2; };

// A phase's weight matrix is cut into units: 16 output rows x kchunk input columns.
// unit u -> k-split ks = u / n_tiles, tile = u % n_tiles.
struct PhaseGeom { int n_tiles, KS, kchunk, n_units; };

struct RoundArgs {
  // drafter
  const LayerW* layers;
  const __nv_bfloat16 *embed, *lm_head, *final_norm;
  const float *rope_cos, *rope_sin;
  int L, d, F, H, Hkv, hd, V, cap, qkv_w;
  float eps, attn_scale;
  PhaseGeom geom[5];
  int slot_bytes, n_ring, act_bytes, split_len;
  // round
  int R, B, m, G, greedy;
  const int* kv_len;                    // [R] committed lengths (constant during the round)
  const int* pending;                   // [B][3]
  __nv_bfloat16 *kc, *vc;               // [R][L][Hkv][cap][hd]
  // activations exchanged through L2
  float *xa, *x1;                       // [8][d] residual before / after the attention block
  float *pq, *po, *pd;                  // split-K partial sums [KS][8][width]
  float *mid, *attn_out;                // [8][F], [8][H*hd]
  float *part_o, *part_ml;              // attention partials [8][H][max_splits][hd], [..][2]
  int max_splits;
  int* tickets;                         // [8][Hkv]
  // ensemble
  float* logits_own;                    // [G][R][V]
  const float* logits_override;         // or null
  const float* w;                       // [B][m]
  const float* u;                       // [B][G]
  float *qk, *q;                        // [B][G][m][V], [B][G][V]
  uint32_t* rowmax;                     // [G][R]
  unsigned long long* rowsum;           // [G][R]
  unsigned long long* chunk_mass;       // [B][n_chunks]
  ChunkBest* chunk_best;                // [B][n_chunks]
  int n_chunks;
  int *tokens, *out_tokens;             // [B][G]
  // synchronisation / diagnostics
  unsigned* bar;                        // [2] grid barrier counters, used alternately by launches
  int bar_sel;
  int* err;
  unsigned long long* trace;            // optional [G][trace_stride] globaltimer after each barrier
  int trace_stride;
};

// ------------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// global -> shared bulk copy; dst/src 16-byte aligned, bytes a multiple of 16.  No multicast.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, unsigned bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x2(uint32_t (&r)[2], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
__device__ __forceinline__ unsigned ld_acquire_u32(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// ------------------------------------------------------------------------------------------------
// per-CTA state
// ------------------------------------------------------------------------------------------------
struct PSlot { int row, pos, active, tok; };

struct PShared {
  uint64_t full[kPRing];
  float sc[kMaxGroup][kAttnSplitMax];
  float q[kMaxGroup][128];
  float kf[2][128], vf[2][128];
  float red[kPW][kPSlots];
  unsigned long long red64[kPW];
  float bestv[kPW]; int besti[kPW];
  float scale[kPSlots];
  float m_[kMaxGroup], l_[kMaxGroup];
  PSlot slot[kPSlots];
  int lm_src[kPSlots];
  int tok[kPSlots];
  int dead, flag, result, chunk;
  unsigned long long thr, total;
};

// Walks the CTA's units in consumption order: for each step, for each layer QKV, O, GU, DN, then
// the LM head.  Units of a phase are dealt round-robin over the CTAs, continuing where the
// previous phase stopped, so every CTA streams the same number of bytes (+-1 unit).
struct UnitCursor { int step, p, j, off; };
struct UnitRef { int kind, layer, u; };

__device__ __forceinline__ bool next_unit(const RoundArgs& A, int cta, int NC, UnitCursor& c, UnitRef& out) {
  const int n_phase = 4 * A.L + 1;
  while (c.step < A.G) {
    while (c.p < n_phase) {
      const int kind = (c.p == n_phase - 1) ? KIND_LM : (c.p & 3);
      const int n = A.geom[kind].n_units;
      int first = cta - c.off;
      if (first < 0) first += NC;
      const int u = first + c.j * NC;
      if (u < n) { out.kind = kind; out.layer = c.p >> 2; out.u = u; c.j++; return true; }
      c.off = (c.off + n) % NC; c.p++; c.j = 0;
    }
    c.step++; c.p = 0; c.j = 0; c.off = 0;
  }
  return false;
}

// Issue the bulk copies of one unit into a ring slot (called by all lanes of warp 0).
__device__ __forceinline__ void issue_unit(const RoundArgs& A, const UnitRef& ur, unsigned char* slot_base,
                                           uint64_t* bar, int lane) {
  const PhaseGeom g = A.geom[ur.kind];
  const int ks = ur.u / g.n_tiles, tile = ur.u - ks * g.n_tiles;
  const unsigned row_bytes = (unsigned)g.kchunk * 2u;
  if (lane == 0) mbar_expect_tx(bar, row_bytes * 16u);
  __syncwarp();
  if (lane < 16) {
    const LayerW* lw = A.layers + ur.layer;
    const __nv_bfloat16* base;
    int row, K;
    if (ur.kind == KIND_QKV) {
      K = A.d; row = tile * 16 + lane;
      const int kvd = A.Hkv * A.hd;
      if (row < A.d) base = lw->wq;
      else if (row < A.d + kvd) { base = lw->wk; row -= A.d; }
      else { base = lw->wv; row -= A.d + kvd; }
    } else if (ur.kind == KIND_O) {
      K = A.H * A.hd; row = tile * 16 + lane; base = lw->wo;
    } else if (ur.kind == KIND_GU) {            // rows 0-7: gate rows, rows 8-15: the matching up rows
      K = A.d; row = tile * 8 + (lane & 7); base = (lane < 8) ? lw->wg : lw->wu;
    } else if (ur.kind == KIND_DN) {
      K = A.F; row = tile * 16 + lane; base = lw->wd;
    } else {
      K = A.d; row = min(tile * 16 + lane, A.V - 1); base = A.lm_head;
    }
    const __nv_bfloat16* src = base + (size_t)row * K + (size_t)ks * g.kchunk;
    bulk_g2s(slot_base + (size_t)lane * (row_bytes + 16u), src, row_bytes, bar);
  }
}

constexpr unsigned kSpinLimit = 1u << 21;

// Bounded wait for a ring slot.  Returns false (and marks the CTA dead) on timeout.
__device__ __forceinline__ bool wait_full(PShared& S, int slot, unsigned parity, int* err) {
  unsigned spins = 0;
  while (!mbar_try_wait(&S.full[slot], parity)) {
    if (++spins > kSpinLimit) { atomicOr(err, PERR_COPY); S.dead = 1; return false; }
    if (spins > 4096) __nanosleep(64);
  }
  return true;
}

// Grid-wide barrier on a monotonically increasing counter.  Returns false if the CTA is dead.
__device__ __forceinline__ bool grid_barrier(PShared& S, unsigned* bar, unsigned target, int* err) {
  __syncthreads();
  if (threadIdx.x == 0 && !S.dead) {
    __threadfence();
    atomicAdd(bar, 1u);
    unsigned spins = 0;
    while ((int)(ld_acquire_u32(bar) - target) < 0) {
      if (++spins > kSpinLimit) { atomicOr(err, PERR_BARRIER); S.dead = 1; break; }
      if (spins > 4096) __nanosleep(64);
    }
    __threadfence();
  }
  __syncthreads();
  return S.dead == 0;
}

__device__ __forceinline__ unsigned long long block_sum_u64_p(unsigned long long v, PShared& S) {
  v = warp_sum_u64(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) S.red64[w] = v;
  __syncthreads();
  unsigned long long t = 0;
#pragma unroll
  for (int i = 0; i < kPW; ++i) t += S.red64[i];
  return t;           // valid in every thread
}

__device__ __forceinline__ void load4_cg(const float* __restrict__ row, int v0, int V, bool vec, float fill,
                                         float (&x)[kPPer]) {
  if (vec && v0 + kPPer <= V) {
    const float4 a = __ldcg(reinterpret_cast<const float4*>(row + v0));
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
  } else {
#pragma unroll
    for (int j = 0; j < kPPer; ++j) x[j] = (v0 + j < V) ? __ldcg(row + v0 + j) : fill;
  }
}
__device__ __forceinline__ void store4(float* __restrict__ row, int v0, int V, bool vec, const float (&x)[kPPer]) {
  if (vec && v0 + kPPer <= V) {
    *reinterpret_cast<float4*>(row + v0) = make_float4(x[0], x[1], x[2], x[3]);
  } else {
#pragma unroll
    for (int j = 0; j < kPPer; ++j) if (v0 + j < V) row[v0 + j] = x[j];
  }
}

// ------------------------------------------------------------------------------------------------
// the kernel
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPT, 1) k_draft_round(const RoundArgs A) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ PShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cta = blockIdx.x, NC = gridDim.x;
  unsigned char* ring = dyn_smem;
  unsigned char* U = dyn_smem + (size_t)A.n_ring * A.slot_bytes;
  __nv_bfloat16* act = reinterpret_cast<__nv_bfloat16*>(U);               // [8][apitch]
  float* cpart = reinterpret_cast<float*>(U + A.act_bytes);               // [2][kPW][128]
  float* s_o = reinterpret_cast<float*>(U);                               // attention: [kPW][grp*hd]
  unsigned* bar = A.bar + A.bar_sel;
  const int kvd = A.Hkv * A.hd, HD = A.H * A.hd, grp = A.H / A.Hkv, half = A.hd >> 1;
  const int R = A.R, B = A.B, m = A.m, G = A.G, V = A.V, d = A.d;

  // ---- set-up -----------------------------------------------------------------------------------
  if (tid == 0) {
    for (int s = 0; s < A.n_ring; ++s) mbar_init(&S.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    S.dead = 0;
  }
  if (cta == 0) {
    for (int i = tid; i < G * R; i += kPT) { A.rowmax[i] = 0u; A.rowsum[i] = 0ull; }
    for (int i = tid; i < kPSlots * A.Hkv; i += kPT) A.tickets[i] = 0;
    if (tid == 0) A.bar[A.bar_sel ^ 1] = 0u;          // the next launch's counter
  }
  __syncthreads();

  UnitCursor pc{0, 0, 0, 0};
  unsigned prod_i = 0, cons_i = 0;
  if (warp == 0) {
    for (int k = 0; k < A.n_ring; ++k) {
      UnitRef ur;
      if (!next_unit(A, cta, NC, pc, ur)) break;
      issue_unit(A, ur, ring + (size_t)k * A.slot_bytes, &S.full[k], lane);
      ++prod_i;
    }
  }
  unsigned bar_target = 0;
  bool alive = true;

#define GRID_SYNC()                                                        \
  do {                                                                     \
    bar_target += (unsigned)NC;                                            \
    alive = grid_barrier(S, bar, bar_target, A.err);                       \
    if (A.trace && cta == 0 && tid == 0 && trace_n < A.trace_stride)       \
      A.trace[(size_t)step * A.trace_stride + trace_n++] = global_timer(); \
    if (!alive) goto drain;                                                \
  } while (0)

  for (int step = 0; step < G; ++step) {
    int trace_n = 0;
    // ---- slot table of the step ------------------------------------------------------------------
    int ns = R;
    if (step == 0) {
      for (int b = 0; b < B; ++b) if (A.pending[b * 3] == 2) ns = 2 * R;
    }
    if (tid < kPSlots) {
      PSlot sl{0, 0, 0, 0};
      if (tid < ns) {
        const int row = tid % R, b = row / m, second = tid >= R;
        const int* pend = A.pending + b * 3;
        sl.row = row;
        if (step == 0) {
          sl.pos = A.kv_len[row] + second;
          sl.tok = pend[1 + second];
          sl.active = second ? (pend[0] == 2) : 1;
        } else {
          sl.pos = A.kv_len[row] + pend[0] + step - 1;
          sl.tok = S.tok[b];
          sl.active = 1;
        }
        if (sl.active && sl.pos >= A.cap) { sl.active = 0; atomicOr(A.err, PERR_KV); }
      }
      S.slot[tid] = sl;
      if (tid < R) {
        const int b = tid / m;
        S.lm_src[tid] = (step == 0 && A.pending[b * 3] == 2) ? R + tid : tid;
      }
    }
    __syncthreads();
    int off = 0;                                    // round-robin offset of the current phase

    for (int phase = 0; phase <= 4 * A.L; ++phase) {
      const int kind = (phase == 4 * A.L) ? KIND_LM : (phase & 3);
      const int layer = phase >> 2;
      const LayerW* lw = A.layers + (kind == KIND_LM ? 0 : layer);
      const PhaseGeom g = A.geom[kind];
      const int apitch = g.kchunk + 8;                       // bf16 elements
      const int n_in = (kind == KIND_LM) ? R : ns;           // activation rows of the phase

      // ---- resolve the phase input (residual + split-K partials), RMSNorm statistics -------------
      float xv[kPSlots][kPXE];
      if (kind == KIND_QKV || kind == KIND_GU || kind == KIND_LM) {
        const int KSp = (kind == KIND_GU) ? A.geom[KIND_O].KS : A.geom[KIND_DN].KS;
        const float* part = (kind == KIND_GU) ? A.po : A.pd;
        const float* basebuf = (kind == KIND_GU) ? A.xa : A.x1;
        float* outbuf = (kind == KIND_QKV) ? A.xa : (kind == KIND_GU ? A.x1 : nullptr);
        const int lo = (int)((long long)cta * d / NC), hi = (int)((long long)(cta + 1) * d / NC);
        float ss[kPSlots];
#pragma unroll
        for (int s = 0; s < kPSlots; ++s) {
          ss[s] = 0.0f;
          if (s >= n_in) continue;
          const int src = (kind == KIND_LM) ? S.lm_src[s] : s;
          const bool act_s = (kind == KIND_LM) ? true : (S.slot[s].active != 0);
#pragma unroll
          for (int i = 0; i < kPXE; ++i) {
            const int e = tid + i * kPT;
            float v = 0.0f;
            if (e < d && act_s) {
              if (kind == KIND_QKV && layer == 0) {
                v = __bfloat162float(A.embed[(size_t)S.slot[s].tok * d + e]);
              } else {
                v = __ldcg(basebuf + (size_t)src * d + e);
                for (int ks = 0; ks < KSp; ++ks) v += __ldcg(part + ((size_t)ks * kPSlots + src) * d + e);
              }
              if (outbuf && e >= lo && e < hi) outbuf[(size_t)s * d + e] = v;
            }
            xv[s][i] = v;
            ss[s] = fmaf(v, v, ss[s]);
          }
        }
#pragma unroll
        for (int s = 0; s < kPSlots; ++s) ss[s] = warp_sum_f32(ss[s]);
        if (lane == 0) {
#pragma unroll
          for (int s = 0; s < kPSlots; ++s) S.red[warp][s] = ss[s];
        }
        __syncthreads();
        if (tid < kPSlots) {
          float tot = 0.0f;
#pragma unroll
          for (int w2 = 0; w2 < kPW; ++w2) tot += S.red[w2][tid];
          S.scale[tid] = 1.0f / sqrtf(tot / (float)d + A.eps);
        }
        __syncthreads();
      }

      // ---- units of this CTA ------------------------------------------------------------------------
      int first = cta - off;
      if (first < 0) first += NC;
      int cur_ks = -1;
      float lm_max = -INFINITY;
      for (int u = first; u < g.n_units; u += NC) {
        const int ks = u / g.n_tiles, tile = u - ks * g.n_tiles;
        if (ks != cur_ks) {
          // stage the activation chunk [n_in][kchunk] as bf16 (matmul inputs are rounded to bf16)
          const int k0 = ks * g.kchunk;
          if (kind == KIND_QKV || kind == KIND_GU || kind == KIND_LM) {
            const __nv_bfloat16* gain = (kind == KIND_QKV) ? lw->n1 : (kind == KIND_GU ? lw->n2 : A.final_norm);
#pragma unroll
            for (int s = 0; s < kPSlots; ++s) {
              if (s >= n_in) continue;
              const float sc = S.scale[s];
#pragma unroll
              for (int i = 0; i < kPXE; ++i) {
                const int e = tid + i * kPT;
                if (e >= k0 && e < k0 + g.kchunk && e < d)
                  act[s * apitch + (e - k0)] = __float2bfloat16_rn(xv[s][i] * sc * __bfloat162float(gain[e]));
              }
            }
          } else {
            const float* src = (kind == KIND_O) ? A.attn_out : A.mid;
            const int stride = (kind == KIND_O) ? HD : A.F;
            const int nvec = g.kchunk >> 2;
            for (int idx = tid; idx < n_in * nvec; idx += kPT) {
              const int s = idx / nvec, j = (idx - s * nvec) << 2;
              const float4 v = __ldcg(reinterpret_cast<const float4*>(src + (size_t)s * stride + k0 + j));
              uint2 pk;
              pk.x = pack_bf16(v.x, v.y); pk.y = pack_bf16(v.z, v.w);
              *reinterpret_cast<uint2*>(act + s * apitch + j) = pk;
            }
          }
          cur_ks = ks;
          __syncthreads();
        }
        const int slot = (int)(cons_i % (unsigned)A.n_ring);
        const unsigned parity = (cons_i / (unsigned)A.n_ring) & 1u;
        const bool landed = wait_full(S, slot, parity, A.err);
        if (__syncthreads_or(!landed)) { alive = false; goto drain; }
        const unsigned char* tile_s = ring + (size_t)slot * A.slot_bytes;
        const uint32_t tpitch = (uint32_t)g.kchunk * 2u + 16u;
        float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
        {
          const uint32_t a_base = smem_u32(tile_s) + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * tpitch + (uint32_t)(lane >> 4) * 16u;
          const uint32_t b_base = smem_u32(act) + (uint32_t)(lane & 7) * (uint32_t)apitch * 2u + (uint32_t)((lane >> 3) & 1) * 16u;
          const int nkb = g.kchunk >> 4;
          for (int kb = warp; kb < nkb; kb += kPW) {
            uint32_t a[4], bfr[2];
            ldsm_x4(a, a_base + (uint32_t)kb * 32u);
            ldsm_x2(bfr, b_base + (uint32_t)kb * 32u);
            mma_bf16(c, a, bfr);
          }
        }
        float* cp = cpart + (size_t)(cons_i & 1u) * (kPW * 128);
        {
          const int gq = lane >> 2, tq = lane & 3;
          float* w0 = cp + warp * 128;
          *reinterpret_cast<float2*>(w0 + gq * 8 + tq * 2) = make_float2(c[0], c[1]);
          *reinterpret_cast<float2*>(w0 + (gq + 8) * 8 + tq * 2) = make_float2(c[2], c[3]);
        }
        __syncthreads();                        // slot fully read, partial tiles complete
        if (warp == 0) {                        // refill the slot that was just released
          UnitRef ur;
          if (next_unit(A, cta, NC, pc, ur)) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue_unit(A, ur, ring + (size_t)slot * A.slot_bytes, &S.full[slot], lane);
            ++prod_i;
          }
        }
        ++cons_i;
        if (tid < 128) {                        // sum the warps' partial tiles, epilogue
          const int r = tid & 15, n = tid >> 4;
          float v = 0.0f;
#pragma unroll
          for (int w2 = 0; w2 < kPW; ++w2) v += cp[w2 * 128 + r * 8 + n];
          if (kind == KIND_GU) {
            const float up = __shfl_down_sync(0xffffffffu, v, 8);
            if (r < 8 && n < n_in && S.slot[n].active)
              A.mid[(size_t)n * A.F + tile * 8 + r] = v / (1.0f + expf(-v)) * up;
          } else if (kind == KIND_LM) {
            const int vi = tile * 16 + r;
            float mx = (vi < V && n < n_in) ? v : -INFINITY;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            lm_max = fmaxf(lm_max, mx);
            if (vi < V && n < n_in) A.logits_own[((size_t)step * R + n) * V + vi] = v;
          } else if (n < n_in && S.slot[n].active) {
            const int o = tile * 16 + r;
            if (kind == KIND_QKV) A.pq[((size_t)ks * kPSlots + n) * A.qkv_w + o] = v;
            else if (kind == KIND_O) A.po[((size_t)ks * kPSlots + n) * d + o] = v;
            else A.pd[((size_t)ks * kPSlots + n) * d + o] = v;
          }
        }
      }
      off = (off + g.n_units) % NC;
      if (kind == KIND_LM && tid < 128 && (tid & 15) == 0 && (tid >> 4) < R && lm_max > -INFINITY)
        atomicMax(A.rowmax + step * R + (tid >> 4), ord_encode(lm_max));
      GRID_SYNC();

      // ---- attention over the rows' caches (after the QKV phase) -----------------------------------
      if (kind == KIND_QKV) {
        const int KSq = A.geom[KIND_QKV].KS;
        const int split_len = A.split_len;
        int total_items = 0;
        for (int s = 0; s < ns; ++s)
          if (S.slot[s].active) total_items += A.Hkv * ((S.slot[s].pos + split_len) / split_len);
        for (int item = cta; item < total_items; item += NC) {
          int s = 0, rem = item, nsplit = 0;
          for (; s < ns; ++s) {
            nsplit = S.slot[s].active ? (S.slot[s].pos + split_len) / split_len : 0;
            if (rem < A.Hkv * nsplit) break;
            rem -= A.Hkv * nsplit;
          }
          if (s >= ns) break;
          const int gk = rem / nsplit, split = rem - gk * nsplit;
          const PSlot si = S.slot[s];
          const int pos = si.pos, n_pos = pos + 1;
          const int p_lo = split * split_len, p_hi = min(p_lo + split_len, n_pos), cnt = p_hi - p_lo;
          const int second = s >= R;
          const int n_fresh = second ? 2 : 1;          // positions whose K,V are produced in this very phase
          // stage q (all heads of the group), fresh k and v: split-K sums, RoPE, bf16 rounding
          for (int idx = tid; idx < grp * half; idx += kPT) {
            const int t = idx / half, i = idx - t * half;
            const int col = (gk * grp + t) * A.hd + i;
            float x1 = 0.0f, x2 = 0.0f;
            for (int ks = 0; ks < KSq; ++ks) {
              const float* pr = A.pq + ((size_t)ks * kPSlots + s) * A.qkv_w + col;
              x1 += __ldcg(pr); x2 += __ldcg(pr + half);
            }
            const float cs = A.rope_cos[(size_t)pos * half + i], sn = A.rope_sin[(size_t)pos * half + i];
            S.q[t][i] = round_bf16(x1 * cs - x2 * sn);
            S.q[t][i + half] = round_bf16(x2 * cs + x1 * sn);
          }
          for (int idx = tid; idx < n_fresh * half; idx += kPT) {
            const int j = idx / half, i = idx - j * half;
            const int sj = s - j * R, pj = pos - j;
            const int col = d + gk * A.hd + i;
            float x1 = 0.0f, x2 = 0.0f;
            for (int ks = 0; ks < KSq; ++ks) {
              const float* pr = A.pq + ((size_t)ks * kPSlots + sj) * A.qkv_w + col;
              x1 += __ldcg(pr); x2 += __ldcg(pr + half);
            }
            const float cs = A.rope_cos[(size_t)pj * half + i], sn = A.rope_sin[(size_t)pj * half + i];
            S.kf[j][i] = round_bf16(x1 * cs - x2 * sn);
            S.kf[j][i + half] = round_bf16(x2 * cs + x1 * sn);
          }
          for (int idx = tid; idx < n_fresh * A.hd; idx += kPT) {
            const int j = idx / A.hd, i = idx - j * A.hd;
            const int sj = s - j * R;
            float x = 0.0f;
            for (int ks = 0; ks < KSq; ++ks) x += __ldcg(A.pq + ((size_t)ks * kPSlots + sj) * A.qkv_w + d + kvd + gk * A.hd + i);
            S.vf[j][i] = round_bf16(x);
          }
          __syncthreads();
          const size_t cache_off = ((((size_t)si.row * A.L + layer) * A.Hkv + gk) * A.cap) * A.hd;
          if (split == nsplit - 1 && tid < A.hd) {       // this item owns the append of its own position
            A.kc[cache_off + (size_t)pos * A.hd + tid] = __float2bfloat16_rn(S.kf[0][tid]);
            A.vc[cache_off + (size_t)pos * A.hd + tid] = __float2bfloat16_rn(S.vf[0][tid]);
          }
          const __nv_bfloat16* kbase = A.kc + cache_off;
          const __nv_bfloat16* vbase = A.vc + cache_off;
          const int LPR = A.hd >> 3;                     // lanes per cache row (8 bf16 per 16-byte load)
          const int PPW = 32 / LPR;
          const int sub = lane % LPR, pgrp = lane / LPR;
          // ---- scores ----
          for (int t0 = 0; t0 < grp; t0 += 4) {          // query heads in groups of 4 (register budget)
            float qf[4][8];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int e = 0; e < 8; ++e) qf[t][e] = (t0 + t < grp) ? S.q[t0 + t][sub * 8 + e] : 0.0f;
            for (int pb = warp * PPW; pb < cnt; pb += kPW * PPW) {
              const int p = pb + pgrp;
              const bool valid = p < cnt;
              uint4 kv = make_uint4(0u, 0u, 0u, 0u);
              if (valid) kv = __ldcg(reinterpret_cast<const uint4*>(kbase + (size_t)(p_lo + p) * A.hd + sub * 8));
              float kf8[8];
              Elem<__nv_bfloat16>::unpack(kv, kf8);
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                float dd = 0.0f;
#pragma unroll
                for (int e = 0; e < 8; ++e) dd = fmaf(kf8[e], qf[t][e], dd);
                for (int o = LPR >> 1; o > 0; o >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, o);
                if (valid && sub == 0 && t0 + t < grp) S.sc[t0 + t][p] = dd * A.attn_scale;
              }
            }
          }
          __syncthreads();
          // scores of the fresh positions come from the staged k, not from the cache
          for (int combo = warp; combo < grp * n_fresh; combo += kPW) {
            const int t = combo / n_fresh, j = combo - t * n_fresh;
            const int pj = pos - j;
            if (pj >= p_lo && pj < p_hi) {
              float dd = 0.0f;
              for (int i = lane; i < A.hd; i += 32) dd = fmaf(S.kf[j][i], S.q[t][i], dd);
              dd = warp_sum_f32(dd);
              if (lane == 0) S.sc[t][pj - p_lo] = dd * A.attn_scale;
            }
          }
          __syncthreads();
          for (int t = warp; t < grp; t += kPW) {
            float mx = -INFINITY;
            for (int p = lane; p < cnt; p += 32) mx = fmaxf(mx, S.sc[t][p]);
            mx = warp_max_f32(mx);
            float sum = 0.0f;
            for (int p = lane; p < cnt; p += 32) { const float e = expf(S.sc[t][p] - mx); S.sc[t][p] = e; sum += e; }
            sum = warp_sum_f32(sum);
            if (lane == 0) { S.m_[t] = mx; S.l_[t] = sum; }
          }
          __syncthreads();
          // ---- P V over the cached positions ----
          const int fresh_lo = pos - (n_fresh - 1);      // absolute positions >= fresh_lo are fresh
          for (int t0 = 0; t0 < grp; t0 += 4) {
            float oacc[4][8];
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int e = 0; e < 8; ++e) oacc[t][e] = 0.0f;
            for (int p = warp * PPW + pgrp; p < cnt; p += kPW * PPW) {
              if (p_lo + p >= fresh_lo) continue;
              const uint4 vv = __ldcg(reinterpret_cast<const uint4*>(vbase + (size_t)(p_lo + p) * A.hd + sub * 8));
              float vf8[8];
              Elem<__nv_bfloat16>::unpack(vv, vf8);
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                if (t0 + t >= grp) break;
                const float pw = S.sc[t0 + t][p];
#pragma unroll
                for (int e = 0; e < 8; ++e) oacc[t][e] = fmaf(pw, vf8[e], oacc[t][e]);
              }
            }
#pragma unroll
            for (int t = 0; t < 4; ++t)
#pragma unroll
              for (int e = 0; e < 8; ++e) {
                float v = oacc[t][e];
                for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                oacc[t][e] = v;
              }
            if (pgrp == 0) {
#pragma unroll
              for (int t = 0; t < 4; ++t) {
                if (t0 + t >= grp) break;
#pragma unroll
                for (int e = 0; e < 8; ++e) s_o[((size_t)warp * grp + t0 + t) * A.hd + sub * 8 + e] = oacc[t][e];
              }
            }
          }
          __syncthreads();
          const bool single = nsplit == 1;
          for (int idx = tid; idx < grp * A.hd; idx += kPT) {
            const int t = idx / A.hd, dd = idx - t * A.hd;
            float v = 0.0f;
#pragma unroll
            for (int w2 = 0; w2 < kPW; ++w2) v += s_o[((size_t)w2 * grp + t) * A.hd + dd];
            for (int j = 0; j < n_fresh; ++j) {
              const int pj = pos - j;
              if (pj >= p_lo && pj < p_hi) v = fmaf(S.sc[t][pj - p_lo], S.vf[j][dd], v);
            }
            const int head = gk * grp + t;
            if (single) {
              A.attn_out[(size_t)s * HD + head * A.hd + dd] = v / S.l_[t];
            } else {
              const size_t pi = ((size_t)s * A.H + head) * A.max_splits + split;
              A.part_o[pi * A.hd + dd] = v;
              if (dd == 0) { A.part_ml[pi * 2] = S.m_[t]; A.part_ml[pi * 2 + 1] = S.l_[t]; }
            }
          }
          if (!single) {
            // the CTA that finishes the last split of a (slot, kv head) merges them in split order
            __threadfence();
            __syncthreads();
            if (tid == 0) S.flag = (atomicAdd(A.tickets + s * A.Hkv + gk, 1) == nsplit - 1);
            __syncthreads();
            if (S.flag) {
              __threadfence();
              for (int idx = tid; idx < grp * A.hd; idx += kPT) {
                const int t = idx / A.hd, dd = idx - t * A.hd;
                const int head = gk * grp + t;
                const size_t base = ((size_t)s * A.H + head) * A.max_splits;
                float M = -INFINITY;
                for (int j = 0; j < nsplit; ++j) M = fmaxf(M, __ldcg(A.part_ml + (base + j) * 2));
                float num = 0.0f, den = 0.0f;
                for (int j = 0; j < nsplit; ++j) {
                  const float f = expf(__ldcg(A.part_ml + (base + j) * 2) - M);
                  num = fmaf(f, __ldcg(A.part_o + (base + j) * A.hd + dd), num);
                  den = fmaf(f, __ldcg(A.part_ml + (base + j) * 2 + 1), den);
                }
                A.attn_out[(size_t)s * HD + head * A.hd + dd] = num / den;
              }
              if (tid == 0) A.tickets[s * A.Hkv + gk] = 0;
            }
          }
          __syncthreads();
        }
        GRID_SYNC();
      }
    }  // phases

    // ---- ensemble: exact softmax of the m rows, weighted average, draw (Algorithm 1 steps 6-7) -----
    {
      const float* lg = A.logits_override ? A.logits_override + (size_t)step * R * V : A.logits_own + (size_t)step * R * V;
      uint32_t* rowmax = A.rowmax + step * R;
      unsigned long long* rowsum = A.rowsum + step * R;
      const bool vec = ((V & 3) == 0) && ((reinterpret_cast<uintptr_t>(lg) & 15) == 0);
      const int n_chunks = A.n_chunks;
      if (A.logits_override) {                        // the maxima gathered by the LM head belong to other logits
        if (cta == 0 && tid < R) rowmax[tid] = 0u;
        GRID_SYNC();
        for (int item = cta; item < R * n_chunks; item += NC) {
          const int row = item / n_chunks, ch = item - row * n_chunks;
          float a[kPPer];
          load4_cg(lg + (size_t)row * V, ch * kChunk + tid * kPPer, V, vec, -INFINITY, a);
          float mx = fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
          mx = warp_max_f32(mx);
          if (lane == 0 && mx > -INFINITY) atomicMax(rowmax + row, ord_encode(mx));
        }
        GRID_SYNC();
      }
      for (int item = cta; item < R * n_chunks; item += NC) {
        const int row = item / n_chunks, ch = item - row * n_chunks;
        const int v0 = ch * kChunk + tid * kPPer;
        const float mx = ord_decode(__ldcg(rowmax + row));
        float a[kPPer];
        load4_cg(lg + (size_t)row * V, v0, V, vec, -INFINITY, a);
        unsigned long long sm = 0;
#pragma unroll
        for (int j = 0; j < kPPer; ++j) if (v0 + j < V) sm += mass_of(xexp(__fsub_rn(a[j], mx)));
        sm = block_sum_u64_p(sm, S);
        if (tid == 0 && sm) atomicAdd(rowsum + row, sm);
      }
      GRID_SYNC();
      for (int item = cta; item < B * n_chunks; item += NC) {
        const int b = item / n_chunks, ch = item - b * n_chunks;
        const int v0 = ch * kChunk + tid * kPPer;
        float acc[kPPer];
        float* qk_b = A.qk + ((size_t)b * G + step) * m * V;
        for (int k = 0; k < m; ++k) {
          const int row = b * m + k;
          const float mx = ord_decode(__ldcg(rowmax + row));
          const float Sn = norm_of(__ldcg(rowsum + row));
          const float wk = A.w[row];
          float a[kPPer];
          load4_cg(lg + (size_t)row * V, v0, V, vec, -INFINITY, a);
#pragma unroll
          for (int j = 0; j < kPPer; ++j) {
            a[j] = __fdiv_rn(xexp(__fsub_rn(a[j], mx)), Sn);
            const float t = __fmul_rn(wk, a[j]);
            acc[j] = (k == 0) ? t : __fadd_rn(acc[j], t);
          }
          store4(qk_b + (size_t)k * V, v0, V, (V & 3) == 0, a);
        }
        store4(A.q + ((size_t)b * G + step) * V, v0, V, (V & 3) == 0, acc);
        if (!A.greedy) {
          unsigned long long sm = 0;
#pragma unroll
          for (int j = 0; j < kPPer; ++j) if (v0 + j < V) sm += mass_of(acc[j]);
          sm = block_sum_u64_p(sm, S);
          if (tid == 0) A.chunk_mass[(size_t)b * n_chunks + ch] = sm;
        } else {
          float bv = -1.0f; int bi = 0x7fffffff;
#pragma unroll
          for (int j = 0; j < kPPer; ++j) if (v0 + j < V && acc[j] > bv) { bv = acc[j]; bi = v0 + j; }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          __syncthreads();
          if (lane == 0) { S.bestv[warp] = bv; S.besti[warp] = bi; }
          __syncthreads();
          if (tid == 0) {
            for (int i = 1; i < kPW; ++i)
              if (S.bestv[i] > bv || (S.bestv[i] == bv && S.besti[i] < bi)) { bv = S.bestv[i]; bi = S.besti[i]; }
            A.chunk_best[(size_t)b * n_chunks + ch] = ChunkBest{bv, bi};
          }
        }
      }
      GRID_SYNC();
      // every CTA locates the drawn token itself (the next step's embedding gather needs it)
      for (int b = 0; b < B; ++b) {
        if (A.greedy) {
          float bv = -1.0f; int bi = 0x7fffffff;
          for (int c2 = tid; c2 < n_chunks; c2 += kPT) {
            ChunkBest cb;
            *reinterpret_cast<unsigned long long*>(&cb) =
                __ldcg(reinterpret_cast<const unsigned long long*>(A.chunk_best + (size_t)b * n_chunks + c2));
            if (cb.val > bv || (cb.val == bv && cb.idx < bi)) { bv = cb.val; bi = cb.idx; }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
            if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
          }
          __syncthreads();
          if (lane == 0) { S.bestv[warp] = bv; S.besti[warp] = bi; }
          __syncthreads();
          if (tid == 0) {
            for (int i = 1; i < kPW; ++i)
              if (S.bestv[i] > bv || (S.bestv[i] == bv && S.besti[i] < bi)) { bv = S.bestv[i]; bi = S.besti[i]; }
            S.tok[b] = bi;
          }
          __syncthreads();
          continue;
        }
        const unsigned long long* cm = A.chunk_mass + (size_t)b * n_chunks;
        if (tid == 0) {
          unsigned long long T = 0;
          for (int c2 = 0; c2 < n_chunks; ++c2) T += __ldcg(cm + c2);
          S.result = 0x7fffffff;
          if (T == 0ull) { atomicOr(A.err, 1); S.chunk = -1; }
          else {
            const unsigned long long thr = draw_threshold(A.u[b * G + step], T);
            int c2 = 0;
            unsigned long long pre = 0;
            for (; c2 < n_chunks - 1; ++c2) { const unsigned long long nx = pre + __ldcg(cm + c2); if (nx > thr) break; pre = nx; }
            S.chunk = c2; S.thr = thr - pre;
          }
        }
        __syncthreads();
        const int chunk = S.chunk;
        if (chunk >= 0) {
          const unsigned long long thr = S.thr;
          const float* qrow = A.q + ((size_t)b * G + step) * V;
          const int v0 = chunk * kChunk + tid * kPPer;
          float a[kPPer];
          load4_cg(qrow, v0, V, (V & 3) == 0, 0.0f, a);
          unsigned long long mloc[kPPer], tsum = 0;
#pragma unroll
          for (int j = 0; j < kPPer; ++j) { mloc[j] = (v0 + j < V) ? mass_of(a[j]) : 0ull; tsum += mloc[j]; }
          unsigned long long incl = tsum;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += t;
          }
          if (lane == 31) S.red64[warp] = incl;
          __syncthreads();
          unsigned long long wpre = 0;
          for (int i = 0; i < warp; ++i) wpre += S.red64[i];
          unsigned long long run = wpre + incl - tsum;
          if (run <= thr) {
#pragma unroll
            for (int j = 0; j < kPPer; ++j) {
              run += mloc[j];
              if (run > thr && mloc[j] != 0ull) { atomicMin(&S.result, v0 + j); break; }
            }
          }
          __syncthreads();
        }
        if (tid == 0) {
          int y = S.result;
          if (y == 0x7fffffff) { if (chunk >= 0) atomicOr(A.err, 2); y = 0; }
          S.tok[b] = y;
        }
        __syncthreads();
      }
      if (cta == 0 && tid < B) {
        A.tokens[tid * G + step] = S.tok[tid];
        if (A.out_tokens) A.out_tokens[tid * G + step] = S.tok[tid];
      }
      __syncthreads();
    }
  }  // steps
#undef GRID_SYNC
  return;

drain:
  // a wait ran out: let the copies already issued land before the shared memory is released
  if (tid == 0) {
    for (unsigned k = cons_i; k < prod_i; ++k) {
      const int slot = (int)(k % (unsigned)A.n_ring);
      const unsigned parity = (k / (unsigned)A.n_ring) & 1u;
      unsigned spins = 0;
      while (!mbar_try_wait(&S.full[slot], parity) && ++spins < kSpinLimit) __nanosleep(64);
    }
  }
  __syncthreads();
}

}  // namespace tabed
