// Weight-shared projections for MANY rows (batched serving: 32 requests x 3 inputs = 96 shared-weight
// rows, 192 slots when every request feeds two pending tokens): out[slot][o] = sum_k W[o][k] act[slot][k]
// on the 5th-generation tensor cores.  With ~100 rows per weight byte this is a real dense
// contraction (the SIMT path re-reads the weights once per 8 rows), so it runs as tcgen05.mma with
// the accumulator in tensor memory:
//
//   D[128 weight rows][N slots] += A[128][16] * B[N][16]^T     (kind::f16, bf16 inputs, fp32 accumulate)
//
// * A work unit is (tile of 128 weight rows, range of input columns); split-K over the input
//   dimension gives >= one unit per SM even for the 768-row projections.  Units write fp32 partial
//   sums [k-split][slot][row]; the consumer of the projection adds them in k-split order (deterministic).
// * Operands reach shared memory by bulk asynchronous copies (cp.async.bulk + mbarrier), three stages of
//   128 input columns.  Both operands are stored in global memory already in the tensor core's canonical
//   K-major, no-swizzle layout (8 rows x 16 bytes core matrices), so a stage is two contiguous copies and
//   needs no tensor map: the weights are re-laid once at set-up (k_pack_tc), the activations by the kernel
//   that normalises and rounds them (k_prep_act).
// * One thread issues the copies and the MMAs; tcgen05.commit releases a stage / signals the epilogue;
//   eight warps read the accumulator with tcgen05.ld (warps w and w + 4 own TMEM lanes 32w..32w+31, half of the columns each) and store
//   coalesced rows.  Every wait is bounded; on a timeout the CTA sets an error bit, drains and frees TMEM.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "round_kernel.cuh"   // PTX wrappers: mbarrier, bulk copy

namespace tabed {

constexpr int kTcM = 128;          // weight rows per tile (MMA M)
constexpr int kTcKC = 128;         // input columns per pipeline stage
constexpr int kTcStages = 3;        // pipeline stages (2 when more than 128 slots share the shared memory)
constexpr int kTcMaxStages = 8;
constexpr int kTcThreads = 256;      // eight warps: warps w and w + 4 read the same 32 accumulator lanes, half of the columns each
constexpr int kPrefillChunk = 256;        // positions of one row prefilled as slots of one weight pass
constexpr int kTcMaxN = 256;       // slots per launch (MMA N is their count rounded up to 16)
__host__ __device__ inline int tc_stages(int n_pad) { return n_pad > 128 ? 2 : kTcStages; }

// Canonical K-major no-swizzle operand block of `rows` rows x kTcKC columns (bf16):
// element (r, k) at ((k/8) * (rows/8) + r/8) * 128 + (r%8) * 16 + (k%8) * 2 bytes.
__host__ __device__ inline size_t tc_block_bytes(int rows) { return (size_t)rows * kTcKC * 2; }

struct TcGemmArgs {
  const unsigned char* a_packed;   // [m_tiles][k_chunks] blocks of 128 rows
  const unsigned char* b_packed;   // [k_chunks] blocks of n_pad rows
  float* partial;                  // [ks] slabs of `slab` floats; slab layout [slot][rows_total], first slot of this launch at +0
  size_t slab;                     // floats between k-split slabs
  const SlotDesc* slots;           // optional: the launch returns at once when none of its slots is active
  int rows_total;                  // output rows of the projection (multiple of 128 after padding in a_packed)
  int rows_valid;                  // rows actually stored
  int n_pad, n_slots;              // MMA N (multiple of 16) / slots stored
  int k_chunks;                    // chunks of 128 columns over the whole input dimension
  int ks;                          // k-splits; unit (m_tile, split) covers chunks [split*cps, min((split+1)*cps, k_chunks))
  int cps;                         // chunks per split
  int kc;                          // input columns per pipeline stage: 128 (a whole block) or 64 (half a block: a block's
                                   // 16-byte column groups are its outer index, so half of it is contiguous too)
  int n_stages;                    // pipeline stages, <= kTcMaxStages
  int* err;
};

__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  // shared-memory matrix descriptor: start address, leading (K) and stride (row group) byte offsets in
  // 16-byte units, descriptor version 1 (bits 46-47), no swizzle (bits 61-63 = 0)
  return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}

__device__ __forceinline__ bool tc_wait(uint64_t* bar, unsigned parity, int* err) {
  unsigned spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++spins > (1u << 20)) { atomicOr(err, PERR_COPY); return false; }
    if (spins > 2048) __nanosleep(64);
  }
  return true;
}

// grid (m_tiles * ks), block 128, dynamic shared memory kTcStages * (A block + B block) + 1 KB
__global__ void __launch_bounds__(kTcThreads, 1) k_gemm_tc(const TcGemmArgs G) {
  extern __shared__ __align__(1024) unsigned char tc_smem[];
  __shared__ uint64_t s_full[kTcMaxStages], s_empty[kTcMaxStages], s_done;
  __shared__ uint32_t s_tmem;
  __shared__ int s_bad;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  pdl_trigger();
  const int m_tile = blockIdx.x / G.ks, split = blockIdx.x - m_tile * G.ks;
  // the CTA's range of the input dimension in units of one stage (kc columns); a_bytes, b_bytes = one stage of each operand
  const int per_chunk = kTcKC / G.kc;
  const int c_lo = split * G.cps, c_hi = min(c_lo + G.cps, G.k_chunks), n_ch = (c_hi - c_lo) * per_chunk;
  const size_t a_bytes = tc_block_bytes(kTcM) / per_chunk, b_bytes = tc_block_bytes(G.n_pad) / per_chunk;
  const int n_stages = G.n_stages;
  const uint32_t tmem_cols = G.n_pad <= 32 ? 32u : (G.n_pad <= 64 ? 64u : (G.n_pad <= 128 ? 128u : 256u));

  if (tid == 0) {
    for (int s = 0; s < n_stages; ++s) { mbar_init(&s_full[s], 1); mbar_init(&s_empty[s], 1); }
    mbar_init(&s_done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_bad = 0;
  }
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = s_tmem;
  const unsigned char* a_src = G.a_packed + ((size_t)m_tile * G.k_chunks + c_lo) * tc_block_bytes(kTcM);
  const unsigned char* b_src = G.b_packed + (size_t)c_lo * tc_block_bytes(G.n_pad);
  const int pre = n_ch < n_stages ? n_ch : n_stages;
  // The weights do not depend on the kernels before this one: their first stages are requested before
  // the wait on those kernels (transaction bytes announced without an arrival, so a stage's barrier
  // cannot complete before its activations have been requested too).
  if (tid == 0) {
    for (int c = 0; c < pre; ++c) {
      asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_full[c])), "r"((unsigned)a_bytes) : "memory");
      bulk_g2s(tc_smem + (size_t)c * (a_bytes + b_bytes), a_src + (size_t)c * a_bytes, (unsigned)a_bytes, &s_full[c]);
    }
  }
  pdl_wait();
  {
    int any = 1;
    if (G.slots) {
      any = 0;
      for (int s = tid; s < G.n_slots; s += kTcThreads) any |= G.slots[s].active;
    }
    if (!__syncthreads_or(any)) {
      // nobody needs this pass: let the weight copies land, give the tensor memory back, leave
      if (tid == 0) {
        for (int c = 0; c < pre; ++c) {
          mbar_expect_tx(&s_full[c], 0u);
          unsigned spins = 0;
          while (!mbar_try_wait(&s_full[c], 0) && ++spins < (1u << 20)) __nanosleep(32);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncthreads();
      if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
      return;
    }
  }

  if (tid == 0 && n_ch > 0) {
    // instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, N and M
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(G.n_pad >> 3) << 17) | ((uint32_t)(kTcM >> 4) << 24);
    bool ok = true;
    for (int c = 0; c < pre; ++c) {
      mbar_expect_tx(&s_full[c], (unsigned)b_bytes);
      bulk_g2s(tc_smem + (size_t)c * (a_bytes + b_bytes) + a_bytes, b_src + (size_t)c * b_bytes, (unsigned)b_bytes, &s_full[c]);
    }
    int issued = pre;
    for (int c = 0; c < n_ch && ok; ++c) {
      const int s = c % n_stages;
      ok = tc_wait(&s_full[s], (unsigned)(c / n_stages) & 1u, G.err);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t a_s = smem_u32(tc_smem + (size_t)s * (a_bytes + b_bytes));
      const uint32_t b_s = a_s + (uint32_t)a_bytes;
      const uint32_t a_lbo = (kTcM / 8) * 128, b_lbo = (uint32_t)(G.n_pad / 8) * 128;
#pragma unroll 1
      for (int j = 0; j < G.kc / 16; ++j) {
        const uint64_t da = tc_smem_desc(a_s + (uint32_t)j * 2u * a_lbo, a_lbo, 128u);
        const uint64_t db = tc_smem_desc(b_s + (uint32_t)j * 2u * b_lbo, b_lbo, 128u);
        const uint32_t acc = (c > 0 || j > 0) ? 1u : 0u;
        asm volatile(
            "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
            " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
            ::"r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(acc) : "memory");
      }
      // the stage may be refilled once these MMAs have read it
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_empty[s])) : "memory");
      if (issued < n_ch) {
        ok = tc_wait(&s_empty[s], (unsigned)(c / n_stages) & 1u, G.err);
        if (!ok) break;
        unsigned char* st = tc_smem + (size_t)s * (a_bytes + b_bytes);
        mbar_expect_tx(&s_full[s], (unsigned)(a_bytes + b_bytes));
        bulk_g2s(st, a_src + (size_t)issued * a_bytes, (unsigned)a_bytes, &s_full[s]);
        bulk_g2s(st + a_bytes, b_src + (size_t)issued * b_bytes, (unsigned)b_bytes, &s_full[s]);
        ++issued;
      }
    }
    if (ok) asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_done)) : "memory");
    else {
      s_bad = 1;
      // let the copies in flight land before the shared memory is released
      for (int s = 0; s < n_stages; ++s) {
        unsigned spins = 0;
        while (!mbar_try_wait(&s_full[s], 0) && !mbar_try_wait(&s_full[s], 1) && ++spins < (1u << 16)) __nanosleep(64);
      }
    }
  }
  __syncwarp();
  bool done_ok = true;
  if (n_ch > 0) {
    // everybody waits for the accumulator (or for the issuing thread to give up)
    unsigned spins = 0;
    while (!mbar_try_wait(&s_done, 0)) {
      if (*(volatile int*)&s_bad) { done_ok = false; break; }
      if (++spins > (1u << 21)) { atomicOr(G.err, PERR_COPY); done_ok = false; break; }
      if (spins > 2048) __nanosleep(64);
    }
  }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  if (done_ok) {
    const int lq = warp & 3;                                        // the warp's quarter of the 128 accumulator lanes
    const int row = m_tile * kTcM + lq * 32 + lane;
    float* out = G.partial + (size_t)split * G.slab + row;
    // the warp's columns: the first or the second half of the groups of 16
    const int n16 = G.n_pad >> 4, c_begin = (warp >> 2) ? ((n16 + 1) >> 1) << 4 : 0, c_end = (warp >> 2) ? G.n_pad : ((n16 + 1) >> 1) << 4;
    // two loads of 16 columns in flight: the next one is requested before the current one is stored
    auto ld16 = [&](uint32_t (&v)[16], int c0) {
      const uint32_t taddr = tmem + ((uint32_t)(lq * 32) << 16) + (uint32_t)c0;
      asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                   : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                     "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                   : "r"(taddr));
    };
    auto st16 = [&](const uint32_t (&v)[16], int c0) {
      if (row < G.rows_valid) {
#pragma unroll
        for (int j = 0; j < 16; ++j)
          if (c0 + j < G.n_slots) out[(size_t)(c0 + j) * G.rows_total] = __uint_as_float(v[j]);
      }
    };
    if (n_ch > 0 && c_begin < c_end) {
      uint32_t va[16], vb[16];
      ld16(va, c_begin);
#pragma unroll 1
      for (int c0 = c_begin; c0 < c_end; c0 += 32) {
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        const bool more = c0 + 16 < c_end;
        if (more) ld16(vb, c0 + 16);
        st16(va, c0);
        if (more) {
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          if (c0 + 32 < c_end) ld16(va, c0 + 32);
          st16(vb, c0 + 16);
        }
      }
    } else if (n_ch == 0) {
      if (row < G.rows_valid)
        for (int c = c_begin; c < min(c_end, G.n_slots); ++c) out[(size_t)c * G.rows_total] = 0.0f;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

// ---- operand packing ------------------------------------------------------------------------------
// Weights [rows][K] (one or two matrices concatenated: rows0 of w0 then rows1 of w1) -> blocks
// [m_tile][k_chunk] in the canonical layout; rows beyond rows0+rows1 and columns beyond K are zero.
// grid (k_chunks, m_tiles), block 256.
__global__ void k_pack_tc(const __nv_bfloat16* __restrict__ w0, int rows0, const __nv_bfloat16* __restrict__ w1, int rows1,
                          const __nv_bfloat16* __restrict__ w2, int rows2, int K, int k_chunks, unsigned char* __restrict__ dst) {
  const int kc = blockIdx.x, mt = blockIdx.y;
  unsigned char* blk = dst + ((size_t)mt * k_chunks + kc) * tc_block_bytes(kTcM);
  for (int idx = threadIdx.x; idx < kTcM * (kTcKC / 8); idx += blockDim.x) {
    const int r = idx % kTcM, k8 = idx / kTcM;
    int row = mt * kTcM + r;
    const int k = kc * kTcKC + k8 * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    const __nv_bfloat16* base = nullptr;
    if (row < rows0) base = w0;
    else if (row < rows0 + rows1) { base = w1; row -= rows0; }
    else if (row < rows0 + rows1 + rows2) { base = w2; row -= rows0 + rows1; }
    if (base && k < K) v = *reinterpret_cast<const uint4*>(base + (size_t)row * K + k);
    *reinterpret_cast<uint4*>(blk + ((size_t)k8 * (kTcM / 8) + (r >> 3)) * 128 + (r & 7) * 16) = v;
  }
}

// Activations fp32 [n][K] (row stride `stride`) -> bf16 blocks [k_chunk] of n_pad rows in the canonical
// layout; optional per-row scale (RMSNorm) and bf16 gain.  Rows >= n and columns >= K are zero.
// grid (k_chunks), block 256.
__global__ void k_prep_act(const float* __restrict__ x, int stride, int n, int n_pad, int K, const float* __restrict__ row_scale,
                           const __nv_bfloat16* __restrict__ gain, unsigned char* __restrict__ dst) {
  pdl_trigger();
  pdl_wait();
  const int kc = blockIdx.x;
  unsigned char* blk = dst + (size_t)kc * tc_block_bytes(n_pad);
  for (int idx = threadIdx.x; idx < n_pad * (kTcKC / 8); idx += blockDim.x) {
    const int r = idx % n_pad, k8 = idx / n_pad;
    const int k = kc * kTcKC + k8 * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < n && k < K) {
      const float4 a = *reinterpret_cast<const float4*>(x + (size_t)r * stride + k);
      const float4 b = *reinterpret_cast<const float4*>(x + (size_t)r * stride + k + 4);
      float f[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      if (row_scale) {
        const float sc = row_scale[r];
#pragma unroll
        for (int j = 0; j < 8; ++j) f[j] = f[j] * sc * __bfloat162float(gain[k + j]);
      }
      v.x = pack_bf16(f[0], f[1]); v.y = pack_bf16(f[2], f[3]); v.z = pack_bf16(f[4], f[5]); v.w = pack_bf16(f[6], f[7]);
    }
    *reinterpret_cast<uint4*>(blk + ((size_t)k8 * (n_pad / 8) + (r >> 3)) * 128 + (r & 7) * 16) = v;
  }
}

// ---- activation preparation for the tensor-core projections ------------------------------------------
// One CTA per slot of the group: x <- base + sum of the previous projection's k-split partials (written
// back when `write_back`), optional RMSNorm (gain != null), bf16 rounding, canonical operand layout.
// src_slot (optional) maps the group's row to the slot whose residual it reads (LM head: last slot of a row).
struct PrepRowArgs {
  float* x; int d;                       // residual stream [slot][d]
  const float* partial; int ks; size_t slab;     // [ks] slabs [slot][d] or null
  const int* src_slot;                   // or null
  const SlotDesc* slots;                 // activity of the slots (null: all active)
  const __nv_bfloat16* gain; float eps;  // RMSNorm gain or null
  int slot0, n, n_pad, write_back;
  unsigned char* dst;                    // [k_chunks] blocks of n_pad rows
};
__global__ void __launch_bounds__(256) k_prep_row(const PrepRowArgs P) {
  pdl_trigger();
  pdl_wait();
  const int r = blockIdx.x, tid = threadIdx.x;
  const int s = P.src_slot ? P.src_slot[P.slot0 + r] : P.slot0 + r;
  if (P.slots && !P.slots[s].active) return;
  __shared__ float red[8];
  __shared__ float s_scale;
  float* xr = P.x + (size_t)s * P.d;
  // resolve 8 consecutive elements: the residual plus the slabs, all requested before any is added (slab order kept)
  auto resolve = [&](int k, float (&f)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(xr + k), b = *reinterpret_cast<const float4*>(xr + k + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    for (int q0 = 0; q0 < P.ks; q0 += 8) {
      float4 c[8], e[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const bool ok = q0 + j < P.ks;
        const float* pp = P.partial + (size_t)(ok ? q0 + j : 0) * P.slab + (size_t)s * P.d + k;
        c[j] = ok ? *reinterpret_cast<const float4*>(pp) : make_float4(0.f, 0.f, 0.f, 0.f);
        e[j] = ok ? *reinterpret_cast<const float4*>(pp + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        if (q0 + j < P.ks) {
          f[0] += c[j].x; f[1] += c[j].y; f[2] += c[j].z; f[3] += c[j].w; f[4] += e[j].x; f[5] += e[j].y; f[6] += e[j].z; f[7] += e[j].w;
        }
      }
    }
  };
  auto emit = [&](int k, const float (&f)[8], float sc) {
    float g[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) g[j] = P.gain ? f[j] * sc * __bfloat162float(P.gain[k + j]) : f[j];
    uint4 v;
    v.x = pack_bf16(g[0], g[1]); v.y = pack_bf16(g[2], g[3]); v.z = pack_bf16(g[4], g[5]); v.w = pack_bf16(g[6], g[7]);
    const int kc = k / kTcKC, k8 = (k % kTcKC) >> 3;
    *reinterpret_cast<uint4*>(P.dst + (size_t)kc * tc_block_bytes(P.n_pad) + ((size_t)k8 * (P.n_pad / 8) + (r >> 3)) * 128 + (r & 7) * 16) = v;
  };
  const bool one_pass = P.d <= 256 * 8;              // every thread owns at most one group of 8: it stays in registers
  float keep[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  float ss = 0.0f;
  // pass 1: resolve, write back, sum of squares.  Thread owns groups of 8 consecutive elements.
  for (int k = tid * 8; k < P.d; k += 256 * 8) {
    float f[8];
    resolve(k, f);
    if (P.write_back && P.ks > 0) {
      *reinterpret_cast<float4*>(xr + k) = make_float4(f[0], f[1], f[2], f[3]);
      *reinterpret_cast<float4*>(xr + k + 4) = make_float4(f[4], f[5], f[6], f[7]);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) { ss = fmaf(f[j], f[j], ss); keep[j] = f[j]; }
  }
  ss = warp_sum_f32(ss);
  if ((tid & 31) == 0) red[tid >> 5] = ss;
  __syncthreads();
  if (tid == 0) {
    float tot = 0.0f;
    for (int w = 0; w < 8; ++w) tot += red[w];
    s_scale = P.gain ? 1.0f / sqrtf(tot / (float)P.d + P.eps) : 1.0f;
  }
  __syncthreads();
  const float sc = s_scale;
  // pass 2: scale, round, store 16-byte pieces of the canonical layout (long rows: resolved again, the values are in L1/L2)
  if (one_pass) {
    if (tid * 8 < P.d) emit(tid * 8, keep, sc);
  } else {
    for (int k = tid * 8; k < P.d; k += 256 * 8) {
      float f[8];
      if (P.write_back && P.ks > 0) {
        const float4 a = *reinterpret_cast<const float4*>(xr + k), b = *reinterpret_cast<const float4*>(xr + k + 4);
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
      } else {
        resolve(k, f);
      }
      emit(k, f, sc);
    }
  }
}

// Gated product for the down projection from the gate|up projection's partials:
// mid[s][f] = SiLU(sum_q pg[q][s][f]) * (sum_q pg[q][s][F + f]), rounded to bf16, canonical layout.
// grid (k_chunks of F, slots of the group), block 16 (one thread per 8 columns of the chunk).
__global__ void k_swiglu_prep(const float* __restrict__ partial, int ks, size_t slab, int F, const SlotDesc* __restrict__ slots,
                              int slot0, int n_pad, unsigned char* __restrict__ dst) {
  pdl_trigger();
  pdl_wait();
  const int kc = blockIdx.x, r = blockIdx.y, k8 = threadIdx.x;
  const int s = slot0 + r;
  if (slots && !slots[s].active) return;
  const int f0 = kc * kTcKC + k8 * 8;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (f0 < F) {
    float g[8] = {0, 0, 0, 0, 0, 0, 0, 0}, u[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int q0 = 0; q0 < ks; q0 += 4) {              // four slabs requested together, added in slab order
      float4 a[4], b[4], c[4], e[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const bool ok = q0 + j < ks;
        const float* pg = partial + (size_t)(ok ? q0 + j : 0) * slab + (size_t)s * (2 * F) + f0;
        const float4 z = make_float4(0.f, 0.f, 0.f, 0.f);
        a[j] = ok ? *reinterpret_cast<const float4*>(pg) : z; b[j] = ok ? *reinterpret_cast<const float4*>(pg + 4) : z;
        c[j] = ok ? *reinterpret_cast<const float4*>(pg + F) : z; e[j] = ok ? *reinterpret_cast<const float4*>(pg + F + 4) : z;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (q0 + j >= ks) continue;
        g[0] += a[j].x; g[1] += a[j].y; g[2] += a[j].z; g[3] += a[j].w; g[4] += b[j].x; g[5] += b[j].y; g[6] += b[j].z; g[7] += b[j].w;
        u[0] += c[j].x; u[1] += c[j].y; u[2] += c[j].z; u[3] += c[j].w; u[4] += e[j].x; u[5] += e[j].y; u[6] += e[j].z; u[7] += e[j].w;
      }
    }
    float m[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) m[j] = g[j] / (1.0f + expf(-g[j])) * u[j];
    v.x = pack_bf16(m[0], m[1]); v.y = pack_bf16(m[2], m[3]); v.z = pack_bf16(m[4], m[5]); v.w = pack_bf16(m[6], m[7]);
  }
  *reinterpret_cast<uint4*>(dst + (size_t)kc * tc_block_bytes(n_pad) + ((size_t)k8 * (n_pad / 8) + (r >> 3)) * 128 + (r & 7) * 16) = v;
}

}  // namespace tabed
