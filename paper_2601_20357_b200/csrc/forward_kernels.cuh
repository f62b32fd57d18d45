// Batched shared-weight decoder step of the drafter M_q (Algorithm 1 step 5; Sec. 4.1
// "Ensemble learning via Batched Inference"): all rows share one set of parameters, so every
// weight byte is read from HBM once per step for all of them.
//
// A step works on "slots": one (row, position, token) each.  A normal step has one slot per row;
// the first step of a round after a fully accepted block has two (both pending tokens go through
// the same weight pass).  Slots of one step live in a device-side table so that no kernel
// argument depends on data the host has not seen.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace tabed {

struct SlotDesc { int row; int pos; int active; int pad; };

// ------------------------------------------------------------------------------------------------
// element helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ float round_bf16(float x) { return __bfloat162float(__float2bfloat16_rn(x)); }

// Programmatic dependent launch (kernels of a chain launched with the stream-serialization attribute):
// pdl_trigger lets the next kernel of the stream be scheduled while this one still runs; pdl_wait blocks
// until every kernel before this one has completed and its writes are visible.  A kernel must not touch
// memory that other kernels write, or that they may still read, before pdl_wait.  Both are no-ops in a
// kernel launched without the attribute.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename T> struct Elem;
template <> struct Elem<float> {
  static constexpr int kPerVec = 4;                      // elements per 16-byte load
  __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[4]) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y); f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
  }
  __device__ static __forceinline__ float load(const float* p) { return *p; }
  __device__ static __forceinline__ void store(float* p, float v) { *p = v; }
  __device__ static __forceinline__ float round(float v) { return v; }
};
template <> struct Elem<__nv_bfloat16> {
  static constexpr int kPerVec = 8;
  __device__ static __forceinline__ void unpack(const uint4& v, float (&f)[8]) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xFFFF0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xFFFF0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xFFFF0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xFFFF0000u);
  }
  __device__ static __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  __device__ static __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
  __device__ static __forceinline__ float round(float v) { return round_bf16(v); }
};

// ------------------------------------------------------------------------------------------------
// step table + embedding gather
// ------------------------------------------------------------------------------------------------
enum StepMode { STEP_ROUND_FIRST = 0, STEP_ROUND_NEXT = 1, STEP_FREE = 2, STEP_PREFILL = 3 };

struct StepArgs {
  int mode, R, m, d, G, step;          // step: index i of the drafting step (ROUND_NEXT)
  const int* kv_len;                   // [R]
  const int* pending;                  // [B][3]
  const int* tokens;                   // [B][G] drafted so far (ROUND_NEXT) / [B] caller tokens (FREE)
  int prefill_row, prefill_off;        // PREFILL: row and offset from its committed length
  const int* prefill_tokens;           // [len] or null
  const float* prefill_embeds;         // [len][d] or null
  SlotDesc* slots;                     // [2R]
  int* last_slot;                      // [R]
  float* x;                            // [2R][d] residual stream
  int* err; int kv_capacity;
};

// grid: number of slots of the step; block 128
template <typename T>
__global__ void k_begin_step(StepArgs A, const T* __restrict__ embed) {
  pdl_trigger();
  pdl_wait();
  const int s = blockIdx.x;
  int row, pos, active = 1, tok = -1;
  const float* src_embed = nullptr;
  if (A.mode == STEP_PREFILL) {                    // slot s = position prefill_off + s of the row's new prefix
    row = A.prefill_row;
    pos = A.kv_len[row] + A.prefill_off + s;
    if (A.prefill_tokens) tok = A.prefill_tokens[A.prefill_off + s];
    else src_embed = A.prefill_embeds + (long long)(A.prefill_off + s) * A.d;
  } else {
    row = s % A.R;
    const int b = row / A.m;
    const int second = s >= A.R;
    const int* pend = A.pending + b * 3;
    if (A.mode == STEP_ROUND_FIRST) {
      const int cnt = pend[0];
      pos = A.kv_len[row] + second;
      tok = pend[1 + second];
      active = second ? (cnt == 2) : 1;
      if (!second && threadIdx.x == 0) A.last_slot[row] = (cnt == 2) ? A.R + row : row;
    } else if (A.mode == STEP_ROUND_NEXT) {
      pos = A.kv_len[row] + pend[0] + A.step - 1;
      tok = A.tokens[b * A.G + A.step - 1];
      if (threadIdx.x == 0) A.last_slot[row] = row;
    } else {
      pos = A.kv_len[row];
      tok = A.tokens[b];
      if (threadIdx.x == 0) A.last_slot[row] = row;
    }
  }
  if (active && pos >= A.kv_capacity) { active = 0; if (threadIdx.x == 0 && A.err) atomicOr(A.err, 4); }
  if (threadIdx.x == 0) A.slots[s] = SlotDesc{row, pos, active, 0};
  if (!active) return;
  float* xo = A.x + (long long)s * A.d;
  if (src_embed) {
    for (int i = threadIdx.x; i < A.d; i += blockDim.x) xo[i] = src_embed[i];
  } else {
    const T* e = embed + (long long)tok * A.d;
    for (int i = threadIdx.x; i < A.d; i += blockDim.x) xo[i] = Elem<T>::load(e + i);
  }
}

// Pooled multimodal drafting input (Sec. 5, "Pooled Multimodal Drafting (P)"): visual tokens on a row-major
// grid_h x grid_w grid, every 2 x 2 block replaced by its average.  The sum of four fp32 values is exact in
// fp64, so the result is the correctly rounded mean.  grid (grid_h/2 * grid_w/2), any block size.
__global__ void k_pool2x2(const float* __restrict__ in, int grid_w, int d, float* __restrict__ out) {
  const int ow = grid_w >> 1;
  const int oi = blockIdx.x / ow, oj = blockIdx.x - oi * ow;
  const float* r0 = in + ((size_t)(2 * oi) * grid_w + 2 * oj) * d;
  const float* r1 = r0 + (size_t)grid_w * d;
  float* o = out + (size_t)blockIdx.x * d;
  for (int i = threadIdx.x; i < d; i += blockDim.x)
    o[i] = (float)((((double)r0[i] + (double)r0[d + i]) + ((double)r1[i] + (double)r1[d + i])) * 0.25);
}

// advance committed lengths by one (STEP_FREE: all rows; STEP_PREFILL handled on the host side
// by a single add at the end)
__global__ void k_advance_len(int* kv_len, int R, int row_only, int by) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  if (row_only >= 0 && r != row_only) return;
  kv_len[r] += by;
}

// ------------------------------------------------------------------------------------------------
// K-a: weight-shared projection  out[slot][o] = sum_i W[o][i] * in[slot][i]
//   prologue : optional RMSNorm (gain), optional bf16 rounding of the matmul input; input rows of
//              this CTA's slot chunk are staged once in shared memory as fp32
//   main     : one warp per group of RPW output rows, 128-bit weight loads, NS accumulators per
//              row (one per slot of the chunk), warp-shuffle reduction
//   epilogue : EPI_STORE out = acc; EPI_RESID out += acc; EPI_SWIGLU out = SiLU(acc_gate)*acc_up
// grid (ctas, slot chunks).
// ------------------------------------------------------------------------------------------------
enum { EPI_STORE = 0, EPI_RESID = 1, EPI_SWIGLU = 2 };

struct GemvArgs {
  const void* W0; const void* W1; const void* W2;   // up to three [rows_i][K] matrices, outputs concatenated
  int rows0, rows1, rows2;
  int K;
  const float* in; int in_stride;                   // [slot][K]
  const int* src_slot;                              // optional: input slot of local row j is src_slot[base + j]
  const void* gain; float eps;                      // RMSNorm gain [K] (null: no norm)
  float* out; int out_stride;                       // [slot][rows0+rows1+rows2]  (SWIGLU: [slot][rows0])
  const SlotDesc* slots; int n_slots;               // activity of the step's slots (null: all active)
  uint32_t* rowmax_enc;                             // optional: per-output-slot running max of out (LM head)
};

constexpr int kGemvWarps = 8;
constexpr int kGemvThreads = kGemvWarps * 32;

template <typename T, int NS, int RPW, int EPI, bool ROUND_IN>
__global__ void __launch_bounds__(kGemvThreads) k_gemv(GemvArgs A) {
  extern __shared__ __align__(16) float xs[];          // [NS][K]
  __shared__ float red[kGemvWarps];
  constexpr int EL = Elem<T>::kPerVec;
  const int K = A.K;
  const int slot_base = blockIdx.y * NS;
  const int ns = min(NS, A.n_slots - slot_base);
  if (A.slots) {
    bool any = false;
    for (int j = 0; j < ns; ++j) any |= (A.slots[slot_base + j].active != 0);
    if (!any) return;
  }
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // ---- prologue: stage (normalised, rounded) inputs ----
  for (int j = 0; j < NS; ++j) {
    float* xj = xs + (long long)j * K;
    if (j >= ns) { for (int i = tid; i < K; i += kGemvThreads) xj[i] = 0.0f; continue; }
    const int src = A.src_slot ? A.src_slot[slot_base + j] : (slot_base + j);
    const float* xin = A.in + (long long)src * A.in_stride;
    float scale = 1.0f;
    if (A.gain) {
      float ss = 0.0f;
      for (int i = tid; i < K; i += kGemvThreads) { const float v = xin[i]; ss = fmaf(v, v, ss); }
      ss = warp_sum_f32(ss);
      __syncthreads();
      if (lane == 0) red[warp] = ss;
      __syncthreads();
      float tot = 0.0f;
#pragma unroll
      for (int w = 0; w < kGemvWarps; ++w) tot += red[w];
      scale = 1.0f / sqrtf(tot / (float)K + A.eps);
    }
    const T* g = reinterpret_cast<const T*>(A.gain);
    for (int i = tid; i < K; i += kGemvThreads) {
      float v = xin[i];
      if (A.gain) v = v * scale * Elem<T>::load(g + i);
      xj[i] = ROUND_IN ? Elem<T>::round(v) : v;
    }
  }
  __syncthreads();

  // ---- main loop ----
  const int n_out = (EPI == EPI_SWIGLU) ? A.rows0 : (A.rows0 + A.rows1 + A.rows2);
  const int n_groups = (n_out + RPW - 1) / RPW;
  const int gw = blockIdx.x * kGemvWarps + warp;
  const int GW = gridDim.x * kGemvWarps;
  constexpr int NMAT = (EPI == EPI_SWIGLU) ? 2 : 1;
  for (int g = gw; g < n_groups; g += GW) {
    const int o0 = g * RPW;
    const T* wrow[RPW][NMAT];
#pragma unroll
    for (int r = 0; r < RPW; ++r) {
      int o = min(o0 + r, n_out - 1);
      if (EPI == EPI_SWIGLU) {
        wrow[r][0] = reinterpret_cast<const T*>(A.W0) + (long long)o * K;
        wrow[r][NMAT - 1] = reinterpret_cast<const T*>(A.W1) + (long long)o * K;
      } else {
        const T* base;
        if (o < A.rows0) base = reinterpret_cast<const T*>(A.W0);
        else if (o < A.rows0 + A.rows1) { base = reinterpret_cast<const T*>(A.W1); o -= A.rows0; }
        else { base = reinterpret_cast<const T*>(A.W2); o -= A.rows0 + A.rows1; }
        wrow[r][0] = base + (long long)o * K;
      }
    }
    float acc[RPW][NMAT][NS];
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
      for (int mt = 0; mt < NMAT; ++mt)
#pragma unroll
        for (int j = 0; j < NS; ++j) acc[r][mt][j] = 0.0f;

#pragma unroll 2
    for (int k = lane * EL; k < K; k += 32 * EL) {
      uint4 wv[RPW][NMAT];
#pragma unroll
      for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int mt = 0; mt < NMAT; ++mt)
          wv[r][mt] = __ldg(reinterpret_cast<const uint4*>(wrow[r][mt] + k));
      float xv[NS][EL];
#pragma unroll
      for (int j = 0; j < NS; ++j) {
#pragma unroll
        for (int e4 = 0; e4 < EL / 4; ++e4) {
          const float4 t = *reinterpret_cast<const float4*>(xs + (long long)j * K + k + e4 * 4);
          xv[j][e4 * 4 + 0] = t.x; xv[j][e4 * 4 + 1] = t.y; xv[j][e4 * 4 + 2] = t.z; xv[j][e4 * 4 + 3] = t.w;
        }
      }
#pragma unroll
      for (int r = 0; r < RPW; ++r)
#pragma unroll
        for (int mt = 0; mt < NMAT; ++mt) {
          float wf[EL];
          Elem<T>::unpack(wv[r][mt], wf);
#pragma unroll
          for (int j = 0; j < NS; ++j)
#pragma unroll
            for (int e = 0; e < EL; ++e) acc[r][mt][j] = fmaf(wf[e], xv[j][e], acc[r][mt][j]);
        }
    }
    // ---- reduce + epilogue ----
#pragma unroll
    for (int r = 0; r < RPW; ++r)
#pragma unroll
      for (int mt = 0; mt < NMAT; ++mt)
#pragma unroll
        for (int j = 0; j < NS; ++j) acc[r][mt][j] = warp_sum_f32(acc[r][mt][j]);
    if (lane == 0) {
#pragma unroll
      for (int r = 0; r < RPW; ++r) {
        const int o = o0 + r;
        if (o >= n_out) break;
#pragma unroll
        for (int j = 0; j < NS; ++j) {
          if (j >= ns) break;
          float* dst = A.out + (long long)(slot_base + j) * A.out_stride + o;
          if (EPI == EPI_STORE) {
            *dst = acc[r][0][j];
            if (A.rowmax_enc) atomicMax(A.rowmax_enc + slot_base + j, ord_encode(acc[r][0][j]));
          } else if (EPI == EPI_RESID) {
            *dst = *dst + acc[r][0][j];
          } else {
            const float gt = acc[r][0][j], up = acc[r][NMAT - 1][j];
            *dst = gt / (1.0f + expf(-gt)) * up;
          }
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// RoPE + cache append.  qkv [slot][(H + 2 Hkv) * hd] fp32: q | k | v.  q is rotated in place (and
// rounded to the cache dtype: it is a matmul input), k rotated, k and v rounded and written to the
// cache at the slot's position.  Pairs (i, i + hd/2), angle pos * theta^(-2i/hd) from a table.
// Cache layout [R][L][Hkv][cap][hd].   grid (slots), block 128.
// ------------------------------------------------------------------------------------------------
// part != nullptr: the QKV projection is still ks split-K slabs [ks][slab], summed here in slab order.
// One thread handles one rotation pair (or two v elements) at a time and requests all the slabs' values of it
// before it adds any, so that a slot costs one or two trips to L2, not one per slab.
constexpr int kRopeMaxSlabs = 8;
template <typename T>
__global__ void k_rope_append(float* __restrict__ qkv, const SlotDesc* __restrict__ slots, int H, int Hkv, int hd,
                              const float* __restrict__ rope_cos, const float* __restrict__ rope_sin,
                              T* __restrict__ kc, T* __restrict__ vc, int layer, int L, int cap,
                              const float* __restrict__ part = nullptr, int ks = 0, size_t slab = 0) {
  pdl_trigger();
  pdl_wait();
  const int s = blockIdx.x;
  const SlotDesc sd = slots[s];
  if (!sd.active) return;
  const int half = hd >> 1;
  float* row = qkv + (long long)s * (H + 2 * Hkv) * hd;
  const float* prow = part ? part + (long long)s * (H + 2 * Hkv) * hd : nullptr;
  // values of two columns, the slabs added in slab order
  auto value2 = [&](int col_a, int col_b, float& va, float& vb) {
    if (!prow) { va = row[col_a]; vb = row[col_b]; return; }
    if (ks <= kRopeMaxSlabs) {
      float a[kRopeMaxSlabs], b2[kRopeMaxSlabs];
#pragma unroll
      for (int k = 0; k < kRopeMaxSlabs; ++k) {
        a[k] = k < ks ? prow[(size_t)k * slab + col_a] : 0.0f;
        b2[k] = k < ks ? prow[(size_t)k * slab + col_b] : 0.0f;
      }
      va = 0.0f; vb = 0.0f;
#pragma unroll
      for (int k = 0; k < kRopeMaxSlabs; ++k) if (k < ks) { va += a[k]; vb += b2[k]; }
    } else {
      va = 0.0f; vb = 0.0f;
      for (int k = 0; k < ks; ++k) { va += prow[(size_t)k * slab + col_a]; vb += prow[(size_t)k * slab + col_b]; }
    }
  };
  const float* c = rope_cos + (long long)sd.pos * half;
  const float* sn = rope_sin + (long long)sd.pos * half;
  // q heads and k heads: (H + Hkv) * half pairs
  for (int idx = threadIdx.x; idx < (H + Hkv) * half; idx += blockDim.x) {
    const int head = idx / half, i = idx - head * half;
    float* p = row + head * hd;
    const float ci = c[i], si = sn[i];
    float x1, x2;
    value2(head * hd + i, head * hd + i + half, x1, x2);
    const float r1 = x1 * ci - x2 * si;
    const float r2 = x2 * ci + x1 * si;
    if (head < H) {
      p[i] = Elem<T>::round(r1); p[i + half] = Elem<T>::round(r2);
    } else {
      const int g = head - H;
      T* dst = kc + ((((long long)sd.row * L + layer) * Hkv + g) * cap + sd.pos) * hd;
      Elem<T>::store(dst + i, r1); Elem<T>::store(dst + i + half, r2);
    }
  }
  for (int idx = threadIdx.x; idx < Hkv * half; idx += blockDim.x) {
    const int g = idx / half, i = idx - g * half;
    T* dst = vc + ((((long long)sd.row * L + layer) * Hkv + g) * cap + sd.pos) * hd;
    float v1, v2;
    value2((H + Hkv) * hd + g * hd + i, (H + Hkv) * hd + g * hd + i + half, v1, v2);
    Elem<T>::store(dst + i, v1); Elem<T>::store(dst + i + half, v2);
  }
}

// ------------------------------------------------------------------------------------------------
// K-b: decode attention over separate row caches, split along the sequence.
//   grid (splits, Hkv, slots), block 128.  A CTA handles cache positions
//   [split*SPLIT, min((split+1)*SPLIT, pos+1)) of one slot's row for one KV head and all
//   grp = H/Hkv query heads that share it (each K/V byte is read once per step).
//   Output: un-normalised partial o, running max and sum per (slot, head, split).
// ------------------------------------------------------------------------------------------------
constexpr int kAttnThreads = 128;
constexpr int kAttnSplitMax = 256;
constexpr int kMaxGroup = 8;

template <typename T, int HD>
__global__ void __launch_bounds__(kAttnThreads)
k_attn_partial(const float* __restrict__ qkv, const SlotDesc* __restrict__ slots, int H, int Hkv,
               const T* __restrict__ kc, const T* __restrict__ vc, int layer, int L, int cap, int split_len,
               float* __restrict__ part_o, float* __restrict__ part_ml, int max_splits, float scale) {
  constexpr int EL = Elem<T>::kPerVec;
  constexpr int LPR = HD / EL;                 // lanes per cache row
  constexpr int PPW = 32 / LPR;                // positions per warp pass
  constexpr int NW = kAttnThreads / 32;
  const int s = blockIdx.z, g = blockIdx.y, split = blockIdx.x;
  const SlotDesc sd = slots[s];
  if (!sd.active) return;
  const int n_pos = sd.pos + 1;
  const int p_lo = split * split_len;
  if (p_lo >= n_pos) return;
  const int p_hi = min(p_lo + split_len, n_pos);
  const int cnt = p_hi - p_lo;
  const int grp = H / Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane % LPR, pgrp = lane / LPR;

  __shared__ float sc[kMaxGroup][kAttnSplitMax];
  __shared__ float s_m[kMaxGroup], s_l[kMaxGroup];
  __shared__ float s_o[NW][kMaxGroup][HD];

  const T* kbase = kc + ((((long long)sd.row * L + layer) * Hkv + g) * cap) * HD;
  const T* vbase = vc + ((((long long)sd.row * L + layer) * Hkv + g) * cap) * HD;
  const float* qrow = qkv + (long long)s * (H + 2 * Hkv) * HD + (long long)g * grp * HD;

  for (int t0 = 0; t0 < grp; t0 += kMaxGroup) {
    const int tg = min(kMaxGroup, grp - t0);
    // q fragments of this lane
    float qf[kMaxGroup][EL];
#pragma unroll
    for (int t = 0; t < kMaxGroup; ++t)
#pragma unroll
      for (int e = 0; e < EL; ++e) qf[t][e] = (t < tg) ? qrow[(t0 + t) * HD + sub * EL + e] : 0.0f;
    // ---- scores ----
    for (int pb = warp * PPW; pb < cnt; pb += NW * PPW) {      // warp-uniform trip count
      const int p = pb + pgrp;
      const bool valid = p < cnt;
      uint4 kv = make_uint4(0u, 0u, 0u, 0u);
      if (valid) kv = __ldg(reinterpret_cast<const uint4*>(kbase + (long long)(p_lo + p) * HD + sub * EL));
      float kf[EL];
      Elem<T>::unpack(kv, kf);
#pragma unroll
      for (int t = 0; t < kMaxGroup; ++t) {
        if (t >= tg) break;
        float d = 0.0f;
#pragma unroll
        for (int e = 0; e < EL; ++e) d = fmaf(kf[e], qf[t][e], d);
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
        if (valid && sub == 0) sc[t][p] = d * scale;
      }
    }
    __syncthreads();
    // ---- softmax statistics per head ----
    for (int t = warp; t < tg; t += NW) {
      float mx = -INFINITY;
      for (int p = lane; p < cnt; p += 32) mx = fmaxf(mx, sc[t][p]);
      mx = warp_max_f32(mx);
      float sum = 0.0f;
      for (int p = lane; p < cnt; p += 32) { const float e = expf(sc[t][p] - mx); sc[t][p] = e; sum += e; }
      sum = warp_sum_f32(sum);
      if (lane == 0) { s_m[t] = mx; s_l[t] = sum; }
    }
    __syncthreads();
    // ---- P V ----
    float oacc[kMaxGroup][EL];
#pragma unroll
    for (int t = 0; t < kMaxGroup; ++t)
#pragma unroll
      for (int e = 0; e < EL; ++e) oacc[t][e] = 0.0f;
    for (int p = warp * PPW + pgrp; p < cnt; p += NW * PPW) {
      const uint4 vv = __ldg(reinterpret_cast<const uint4*>(vbase + (long long)(p_lo + p) * HD + sub * EL));
      float vf[EL];
      Elem<T>::unpack(vv, vf);
#pragma unroll
      for (int t = 0; t < kMaxGroup; ++t) {
        if (t >= tg) break;
        const float pw = sc[t][p];
#pragma unroll
        for (int e = 0; e < EL; ++e) oacc[t][e] = fmaf(pw, vf[e], oacc[t][e]);
      }
    }
    // reduce over the position groups of the warp, then over warps
#pragma unroll
    for (int t = 0; t < kMaxGroup; ++t)
#pragma unroll
      for (int e = 0; e < EL; ++e) {
        float v = oacc[t][e];
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        oacc[t][e] = v;
      }
    if (pgrp == 0) {
#pragma unroll
      for (int t = 0; t < kMaxGroup; ++t)
#pragma unroll
        for (int e = 0; e < EL; ++e) s_o[warp][t][sub * EL + e] = oacc[t][e];
    }
    __syncthreads();
    for (int idx = tid; idx < tg * HD; idx += kAttnThreads) {
      const int t = idx / HD, dd = idx - t * HD;
      float v = 0.0f;
#pragma unroll
      for (int w = 0; w < NW; ++w) v += s_o[w][t][dd];
      const int head = g * grp + t0 + t;
      const long long pi = ((long long)s * H + head) * max_splits + split;
      part_o[pi * HD + dd] = v;
      if (dd == 0) { part_ml[pi * 2] = s_m[t]; part_ml[pi * 2 + 1] = s_l[t]; }
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// K-b, bf16 caches, bandwidth-oriented variant: grid (splits, Hkv, slots), block 256.  A CTA handles
// kAttnBwPasses * (8 warps * 32/LPR) positions (128 for head_dim 64) and issues ALL its K and V loads
// (8 x 16 bytes per thread) before it touches any of them, so that one memory round trip covers the
// item and ~4 resident CTAs keep >100 KB per SM in flight.  Output as k_attn_partial.
// ------------------------------------------------------------------------------------------------
constexpr int kAttnBwThreads = 256;
constexpr int kAttnBwPasses = 4;
__host__ __device__ inline int attn_bw_split_len(int hd) { return kAttnBwPasses * (kAttnBwThreads / 32) * (32 / (hd / 8)); }

template <int HD>
__global__ void __launch_bounds__(kAttnBwThreads, 3)
k_attn_split_bf16(const float* __restrict__ qkv, const SlotDesc* __restrict__ slots, int H, int Hkv,
                  const __nv_bfloat16* __restrict__ kc, const __nv_bfloat16* __restrict__ vc, int layer, int L, int cap,
                  float* __restrict__ part_o, float* __restrict__ part_ml, int max_splits, float scale) {
  constexpr int LPR = HD / 8, PPW = 32 / LPR, NW = kAttnBwThreads / 32, PPB = NW * PPW, SPLIT = kAttnBwPasses * PPB;
  const int s = blockIdx.z, g = blockIdx.y, split = blockIdx.x;
  const SlotDesc sd = slots[s];
  if (!sd.active) return;
  const int n_pos = sd.pos + 1, p_lo = split * SPLIT;
  if (p_lo >= n_pos) return;
  const int cnt = min(SPLIT, n_pos - p_lo);
  const int grp = H / Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, sub = lane % LPR, pgrp = lane / LPR;
  extern __shared__ float bw_smem[];
  float* so = bw_smem;                          // [NW][grp][HD] un-normalised outputs of the warps
  float* sm = so + (size_t)NW * grp * HD;       // [NW][grp] running maxima
  float* sl = sm + NW * grp;                    // [NW][grp] sums
  const size_t base = ((((size_t)sd.row * L + layer) * Hkv + g) * cap) * HD;
  uint4 kreg[kAttnBwPasses], vreg[kAttnBwPasses];
#pragma unroll
  for (int ps = 0; ps < kAttnBwPasses; ++ps) {
    const int p = ps * PPB + warp * PPW + pgrp;
    kreg[ps] = make_uint4(0u, 0u, 0u, 0u); vreg[ps] = make_uint4(0u, 0u, 0u, 0u);
    if (p < cnt) {
      kreg[ps] = __ldcs(reinterpret_cast<const uint4*>(kc + base + (size_t)(p_lo + p) * HD + sub * 8));
      vreg[ps] = __ldcs(reinterpret_cast<const uint4*>(vc + base + (size_t)(p_lo + p) * HD + sub * 8));
    }
  }
  const float* qrow = qkv + (size_t)s * (H + 2 * Hkv) * HD + (size_t)g * grp * HD;
  // every warp runs its own softmax over its positions (no block-wide exchange until the end)
#pragma unroll 1
  for (int t = 0; t < grp; ++t) {
    const float4 q0 = *reinterpret_cast<const float4*>(qrow + t * HD + sub * 8);
    const float4 q1 = *reinterpret_cast<const float4*>(qrow + t * HD + sub * 8 + 4);
    const float qf[8] = {q0.x, q0.y, q0.z, q0.w, q1.x, q1.y, q1.z, q1.w};
    float sc[kAttnBwPasses];
    float mx = -INFINITY;
#pragma unroll
    for (int ps = 0; ps < kAttnBwPasses; ++ps) {
      const int p = ps * PPB + warp * PPW + pgrp;
      float kf[8];
      Elem<__nv_bfloat16>::unpack(kreg[ps], kf);
      float d = 0.0f;
#pragma unroll
      for (int e = 0; e < 8; ++e) d = fmaf(kf[e], qf[e], d);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) d += __shfl_xor_sync(0xffffffffu, d, o);
      sc[ps] = (p < cnt) ? d * scale : -INFINITY;
      mx = fmaxf(mx, sc[ps]);
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float oacc[8], sum = 0.0f;
#pragma unroll
    for (int e = 0; e < 8; ++e) oacc[e] = 0.0f;
#pragma unroll
    for (int ps = 0; ps < kAttnBwPasses; ++ps) {
      const float pw = (sc[ps] > -INFINITY) ? expf(sc[ps] - mx) : 0.0f;
      sum += pw;
      float vf[8];
      Elem<__nv_bfloat16>::unpack(vreg[ps], vf);
#pragma unroll
      for (int e = 0; e < 8; ++e) oacc[e] = fmaf(pw, vf[e], oacc[e]);
    }
#pragma unroll
    for (int o = LPR; o < 32; o <<= 1) {
      sum += __shfl_xor_sync(0xffffffffu, sum, o);
#pragma unroll
      for (int e = 0; e < 8; ++e) oacc[e] += __shfl_xor_sync(0xffffffffu, oacc[e], o);
    }
    if (pgrp == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) so[((size_t)warp * grp + t) * HD + sub * 8 + e] = oacc[e];
      if (sub == 0) { sm[warp * grp + t] = mx; sl[warp * grp + t] = sum; }
    }
  }
  __syncthreads();
  // merge the warps in warp order
  for (int idx = tid; idx < grp * HD; idx += kAttnBwThreads) {
    const int t = idx / HD, dd = idx - t * HD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < NW; ++w) M = fmaxf(M, sm[w * grp + t]);
    float v = 0.0f, l = 0.0f;
#pragma unroll
    for (int w = 0; w < NW; ++w) {
      const float mw = sm[w * grp + t];
      const float f = (mw > -INFINITY) ? expf(mw - M) : 0.0f;
      v = fmaf(f, so[((size_t)w * grp + t) * HD + dd], v);
      l = fmaf(f, sl[w * grp + t], l);
    }
    const int head = g * grp + t;
    const long long pi = ((long long)s * H + head) * max_splits + split;
    part_o[pi * HD + dd] = v;
    if (dd == 0) { part_ml[pi * 2] = M; part_ml[pi * 2 + 1] = l; }
  }
}

// merge the splits in fixed order; grid (H, slots), block HD
template <int HD>
__global__ void k_attn_merge(const SlotDesc* __restrict__ slots, int H, int split_len,
                             const float* __restrict__ part_o, const float* __restrict__ part_ml, int max_splits,
                             float* __restrict__ out) {
  const int s = blockIdx.y, head = blockIdx.x, dd = threadIdx.x;
  const SlotDesc sd = slots[s];
  if (!sd.active) return;
  const int n_splits = (sd.pos + 1 + split_len - 1) / split_len;
  const long long base = ((long long)s * H + head) * max_splits;
  float M = -INFINITY;
  for (int j = 0; j < n_splits; ++j) M = fmaxf(M, part_ml[(base + j) * 2]);
  float num = 0.0f, den = 0.0f;
  for (int j = 0; j < n_splits; ++j) {
    const float f = expf(part_ml[(base + j) * 2] - M);
    num = fmaf(f, part_o[(base + j) * HD + dd], num);
    den = fmaf(f, part_ml[(base + j) * 2 + 1], den);
  }
  out[(long long)s * H * HD + head * HD + dd] = num / den;
}

}  // namespace tabed
