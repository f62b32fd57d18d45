// Vocabulary-wide kernels of the round: softmax + ensemble mix + draw (Algorithm 1 steps 6-7),
// verification (Sec. 3 item 3) and deviation / weight update (Sec. 4.1; App. B).
// All are streaming passes over fp32 [rows][V] arrays: 128-bit loads where the row pitch allows,
// warp-shuffle reductions, integer atomics for the cross-CTA sums (exact, order-free).
#pragma once
#include "exact_math.cuh"
#include "forward_kernels.cuh"

namespace tabed {

constexpr int kChunk        = 2048;    // vocabulary elements per CTA
constexpr int kDecThreads   = 256;
constexpr int kPerThread    = kChunk / kDecThreads;   // 8
constexpr int kGridCand     = 11;      // grid policy candidates j = 0..10
constexpr int kMaxInputs   = 8;       // m <= 8
constexpr int kMaxDev       = 11;      // deviations kept per position: 11 grid candidates >= kMaxInputs

// Load this thread's kPerThread consecutive elements of a chunk (zero / fill beyond V).
__device__ __forceinline__ void load8(const float* __restrict__ row, int v0, int V, bool vec, float fill,
                                      float (&x)[kPerThread]) {
  if (vec && v0 + kPerThread <= V) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(row + v0));
    const float4 b = __ldg(reinterpret_cast<const float4*>(row + v0) + 1);
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  } else {
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) x[j] = (v0 + j < V) ? __ldg(row + v0 + j) : fill;
  }
}
__device__ __forceinline__ void store8(float* __restrict__ row, int v0, int V, bool vec,
                                       const float (&x)[kPerThread]) {
  if (vec && v0 + kPerThread <= V) {
    reinterpret_cast<float4*>(row + v0)[0] = make_float4(x[0], x[1], x[2], x[3]);
    reinterpret_cast<float4*>(row + v0)[1] = make_float4(x[4], x[5], x[6], x[7]);
  } else {
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) if (v0 + j < V) row[v0 + j] = x[j];
  }
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* sh) {
  v = warp_sum_u64(v);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
  __syncthreads();
  if (l == 0) sh[w] = v;
  __syncthreads();
  unsigned long long t = 0;
  if (w == 0) {
    t = (l < (int)(blockDim.x >> 5)) ? sh[l] : 0ull;
    t = warp_sum_u64(t);
  }
  return t;   // valid in warp 0
}

// ---- softmax pass 1: row maxima (order-free) -------------------------------------------------
// grid (chunks, rows).  rowmax_enc[row] must be zeroed beforehand.
__global__ void __launch_bounds__(kDecThreads)
k_rowmax(const float* __restrict__ logits, int V, long long row_stride, uint32_t* __restrict__ rowmax_enc) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.y;
  const float* x = logits + (long long)row * row_stride;
  const bool vec = ((V & 3) == 0) && ((row_stride & 3) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
  const int v0 = blockIdx.x * kChunk + threadIdx.x * kPerThread;
  float a[kPerThread];
  load8(x, v0, V, vec, -INFINITY, a);
  float m = a[0];
#pragma unroll
  for (int j = 1; j < kPerThread; ++j) m = fmaxf(m, a[j]);
  m = warp_max_f32(m);
  __shared__ float sh[kDecThreads / 32];
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = sh[0];
    for (int i = 1; i < kDecThreads / 32; ++i) t = fmaxf(t, sh[i]);
    if (t > -INFINITY) atomicMax(rowmax_enc + row, ord_encode(t));
  }
}

// ---- softmax pass 2: integer sum of exp masses -------------------------------------------------
// grid (chunks, rows).  rowsum[row] must be zeroed beforehand.
__global__ void __launch_bounds__(kDecThreads)
k_expsum(const float* __restrict__ logits, int V, long long row_stride,
         const uint32_t* __restrict__ rowmax_enc, unsigned long long* __restrict__ rowsum) {
  pdl_trigger();
  pdl_wait();
  const int row = blockIdx.y;
  const float* x = logits + (long long)row * row_stride;
  const bool vec = ((V & 3) == 0) && ((row_stride & 3) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
  const int v0 = blockIdx.x * kChunk + threadIdx.x * kPerThread;
  const float mx = ord_decode(rowmax_enc[row]);
  float a[kPerThread];
  load8(x, v0, V, vec, -INFINITY, a);
  unsigned long long s = 0;
#pragma unroll
  for (int j = 0; j < kPerThread; ++j)
    if (v0 + j < V) s += mass_of(xexp(__fsub_rn(a[j], mx)));
  __shared__ unsigned long long sh[kDecThreads / 32];
  s = block_sum_u64(s, sh);
  if (threadIdx.x == 0 && s) atomicAdd(rowsum + row, s);
}

// ---- ensemble mix: q^(k) = e/S_k, q = sum_k w_k q^(k), chunk masses (or chunk argmax) -----------
// grid (chunks, B).  logits [B][m][V] (row = b*m + k), w [B][m].
// qk_out [b][..]: pitch qk_req_stride between requests, V between drafters; q_out pitch q_req_stride.
struct ChunkBest { float val; int idx; };

__global__ void __launch_bounds__(kDecThreads)
k_mix(const float* __restrict__ logits, int V, int m, const float* __restrict__ w,
      const uint32_t* __restrict__ rowmax_enc, const unsigned long long* __restrict__ rowsum,
      float* __restrict__ qk_out, long long qk_req_stride,
      float* __restrict__ q_out, long long q_req_stride,
      unsigned long long* __restrict__ chunk_mass, ChunkBest* __restrict__ chunk_best, int n_chunks, int greedy) {
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.y;
  const bool vec = ((V & 3) == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
  const int v0 = blockIdx.x * kChunk + threadIdx.x * kPerThread;
  float acc[kPerThread];
  for (int k = 0; k < m; ++k) {
    const int row = b * m + k;
    const float mx = ord_decode(rowmax_enc[row]);
    const float S = norm_of(rowsum[row]);
    const float wk = w[row];
    float a[kPerThread];
    load8(logits + (long long)row * V, v0, V, vec, -INFINITY, a);
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
      a[j] = __fdiv_rn(xexp(__fsub_rn(a[j], mx)), S);
      const float t = __fmul_rn(wk, a[j]);
      acc[j] = (k == 0) ? t : __fadd_rn(acc[j], t);
    }
    // (vector stores only to 16-byte aligned outputs: the caller's q / qk pointers may be offset views)
    if (qk_out) store8(qk_out + (long long)b * qk_req_stride + (long long)k * V, v0, V,
                       (V & 3) == 0 && (qk_req_stride & 3) == 0 && (reinterpret_cast<uintptr_t>(qk_out) & 15) == 0, a);
  }
  if (q_out) store8(q_out + (long long)b * q_req_stride, v0, V,
                    (V & 3) == 0 && (q_req_stride & 3) == 0 && (reinterpret_cast<uintptr_t>(q_out) & 15) == 0, acc);
  if (!greedy) {
    unsigned long long s = 0;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) if (v0 + j < V) s += mass_of(acc[j]);
    __shared__ unsigned long long sh[kDecThreads / 32];
    s = block_sum_u64(s, sh);
    if (threadIdx.x == 0) chunk_mass[(long long)b * n_chunks + blockIdx.x] = s;
  } else {
    float bv = -1.0f; int bi = 0x7fffffff;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) if (v0 + j < V && acc[j] > bv) { bv = acc[j]; bi = v0 + j; }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __shared__ float shv[kDecThreads / 32];
    __shared__ int shi[kDecThreads / 32];
    if ((threadIdx.x & 31) == 0) { shv[threadIdx.x >> 5] = bv; shi[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int i = 1; i < kDecThreads / 32; ++i)
        if (shv[i] > bv || (shv[i] == bv && shi[i] < bi)) { bv = shv[i]; bi = shi[i]; }
      chunk_best[(long long)b * n_chunks + blockIdx.x] = ChunkBest{bv, bi};
    }
  }
}

// ---- draw: locate the chunk holding the threshold, scan it ---------------------------------------
// Mass source of the scan.
//   SRC_Q     : mass_of(a[v])                         a = q row
//   SRC_RESID : n_accept < G : mass_of(max(0, p_a - q_a)), falling back to mass_of(p_a) when the
//               residual has no mass;  n_accept == G : mass_of(p_G)
struct SelectArgs {
  int V, n_chunks, G, greedy;
  const float* q;   long long q_req_stride;    // [B][..][V]; position pitch = V
  const float* p;                              // [B][G+1][V] (SRC_RESID)
  const int* n_accept;                         // [B]        (SRC_RESID)
  const float* u;   int u_stride;              // u[b*u_stride]
  const unsigned long long* chunk_mass;        // [B][n_chunks]
  const ChunkBest* chunk_best;
  int* out0; int out0_stride;                  // y[b*out0_stride]
  int* out1; int out1_stride;                  // optional second copy
  int* err;
};

__device__ __forceinline__ float resid_val(float p, float q) { return fmaxf(0.0f, __fsub_rn(p, q)); }

template <int SRC>
__global__ void __launch_bounds__(kDecThreads) k_select(SelectArgs A) {
  pdl_trigger();
  pdl_wait();
  const int b = blockIdx.x;
  const int tid = threadIdx.x;
  __shared__ unsigned long long s_thr, s_scan[kDecThreads / 32], s_total;
  __shared__ int s_chunk, s_result, s_fallback;
  const float* arow = nullptr;   // first operand row
  const float* brow = nullptr;   // second operand (residual) or null
  if (SRC == 0) {
    arow = A.q + (long long)b * A.q_req_stride;
  } else {
    const int a = A.n_accept[b];
    arow = A.p + ((long long)b * (A.G + 1) + a) * A.V;
    if (a < A.G) brow = A.q + (long long)b * A.q_req_stride + (long long)a * A.V;
  }
  if (A.greedy) {
    // argmax over chunk bests, lowest index on ties (SRC_RESID greedy: chunk_best holds argmax of p_a)
    float bv = -1.0f; int bi = 0x7fffffff;
    const long long cb_row = (SRC == 0) ? (long long)b : ((long long)b * (A.G + 1) + A.n_accept[b]);
    for (int c = tid; c < A.n_chunks; c += kDecThreads) {
      const ChunkBest cb = A.chunk_best[cb_row * A.n_chunks + c];
      if (cb.val > bv || (cb.val == bv && cb.idx < bi)) { bv = cb.val; bi = cb.idx; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    __shared__ float shv[kDecThreads / 32];
    __shared__ int shi[kDecThreads / 32];
    if ((tid & 31) == 0) { shv[tid >> 5] = bv; shi[tid >> 5] = bi; }
    __syncthreads();
    if (tid == 0) {
      for (int i = 1; i < kDecThreads / 32; ++i)
        if (shv[i] > bv || (shv[i] == bv && shi[i] < bi)) { bv = shv[i]; bi = shi[i]; }
      A.out0[b * A.out0_stride] = bi;
      if (A.out1) A.out1[b * A.out1_stride] = bi;
    }
    return;
  }
  const unsigned long long* cm = A.chunk_mass + (long long)b * A.n_chunks;
  if (tid == 0) {
    unsigned long long T = 0;
    for (int c = 0; c < A.n_chunks; ++c) T += cm[c];
    s_total = T;
    s_fallback = 0;
  }
  __syncthreads();
  if (SRC == 1 && s_total == 0ull) {
    // residual without mass: draw from p_a itself.  Rare; one CTA walks the row.
    brow = nullptr;
    unsigned long long part = 0;
    for (int v = tid; v < A.V; v += kDecThreads) part += mass_of(arow[v]);
    part = block_sum_u64(part, s_scan);
    if (tid == 0) { s_total = part; s_fallback = 1; }
    __syncthreads();
  }
  if (tid == 0) {
    const unsigned long long T = s_total;
    if (T == 0ull) { if (A.err) atomicOr(A.err, 1); s_chunk = -1; }
    else {
      unsigned long long thr = draw_threshold(A.u[b * A.u_stride], T);
      if (s_fallback) {
        s_chunk = -2; s_thr = thr;
      } else {
        int c = 0;
        unsigned long long pre = 0;
        for (; c < A.n_chunks - 1; ++c) { const unsigned long long nx = pre + cm[c]; if (nx > thr) break; pre = nx; }
        s_chunk = c; s_thr = thr - pre;
      }
    }
    s_result = 0x7fffffff;
  }
  __syncthreads();
  int chunk = s_chunk;
  if (chunk == -1) { if (tid == 0) { A.out0[b * A.out0_stride] = 0; if (A.out1) A.out1[b * A.out1_stride] = 0; } return; }
  unsigned long long thr = s_thr;
  const int c_lo = (chunk == -2) ? 0 : chunk;
  const int c_hi = (chunk == -2) ? A.n_chunks : chunk + 1;
  unsigned long long carry = 0;     // mass of the chunks walked so far (fallback walk only)
  for (int c = c_lo; c < c_hi; ++c) {
    const int v0 = c * kChunk + tid * kPerThread;
    unsigned long long mloc[kPerThread];
    unsigned long long tsum = 0;
#pragma unroll
    for (int j = 0; j < kPerThread; ++j) {
      unsigned long long mm = 0;
      if (v0 + j < A.V) {
        const float av = arow[v0 + j];
        mm = mass_of(brow ? resid_val(av, brow[v0 + j]) : av);
      }
      mloc[j] = mm; tsum += mm;
    }
    // exclusive prefix of tsum across the block
    unsigned long long incl = tsum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long t = __shfl_up_sync(0xffffffffu, incl, o);
      if ((tid & 31) >= o) incl += t;
    }
    __syncthreads();
    if ((tid & 31) == 31) s_scan[tid >> 5] = incl;
    __syncthreads();
    unsigned long long wpre = 0;
    for (int i = 0; i < (tid >> 5); ++i) wpre += s_scan[i];
    unsigned long long run = carry + wpre + incl - tsum;
    if (run <= thr) {
#pragma unroll
      for (int j = 0; j < kPerThread; ++j) {
        run += mloc[j];
        if (run > thr && mloc[j] != 0ull) { atomicMin(&s_result, v0 + j); break; }
      }
    }
    unsigned long long ctot = 0;
    for (int i = 0; i < kDecThreads / 32; ++i) ctot += s_scan[i];
    carry += ctot;
    __syncthreads();
    if (s_result != 0x7fffffff) break;
  }
  if (tid == 0) {
    int y = s_result;
    if (y == 0x7fffffff) { if (A.err) atomicOr(A.err, 2); y = 0; }
    A.out0[b * A.out0_stride] = y;
    if (A.out1) A.out1[b * A.out1_stride] = y;
  }
}

// ---- window push, policy, commit (Algorithm 1 steps 2-3; App. B) -----------------------------------
struct PolicyArgs {
  int B, G, m, n_dev, h, policy, tvd, V;
  float tau;                 // temperature of the softmax policy; the constant C of the AdaBoost policy
  const float* u_policy;     // [B][m] uniforms of the random policy
  const int* n_accept;       // [B] accepted tokens of the primary chain
  const int* sib_tok;        // [B] token of the accepted sibling (token tree) or -1
  const int* next_token; const int* tokens;   // [B], [B][G]
  long long* dev;            // [B][G][kMaxDev] deviation sums of the round's verified positions
  long long* ring;           // [B][h][kMaxDev]
  int* ring_head; int* ring_count; long long* pushed;              // [B]
  long long* running;        // [B][kMaxDev]
  float* w;                  // [B][m]
  int* grid_j;               // [B]
  int* kv_len;               // [R] or null (no drafter)
  int* pending;              // [B][3] {cnt, tok0, tok1}
  float* out_w; int* out_argmax;
};

}  // namespace tabed
