// Decode attention over bf16 K,V caches for MANY (slot, KV head) pairs in one launch (the drafting
// step of Algorithm 1 with many rows: every slot attends over its own row's cache).
//
// The work is bound by reading the caches once, so the kernel is built around keeping HBM busy:
//   * a fixed grid of CTAs, each walking a CONTIGUOUS range of the 128-position chunks of all
//     (slot, KV head) caches in (slot, head, position) order;
//   * a chunk of K and of V is one TMA tile each (cp.async.bulk.tensor, 128 rows x 64 dims, 128-byte
//     swizzle), landing in a ring of shared-memory stages several chunks ahead of the arithmetic and
//     signalling an mbarrier: the bytes in flight live in shared memory, not in registers;
//   * the arithmetic runs on the tensor cores (mma.sync m16n8k16) with the cache tile as the A operand
//     (16 positions, resp. 16 dims, as its rows) and the query heads that share the KV head as the 8
//     columns of B, so a tile costs half the mma it would with the (at most 8) heads as the 16 rows;
//     the contraction is far from the tensor roofline, the point is to keep the issue slots free.
//     q and the softmax weights are split into a bf16 head and a bf16 remainder (two products each),
//     K and V are bf16 already, so products are exact to ~2^-17 relative and the sums are fp32;
//   * a warp owns 16 positions of every chunk and carries its own running (max, sum, output) in
//     registers across the chunks of a segment (the part of one cache that this CTA owns).  The
//     warps run free of one another: each waits for a stage's "full" mbarrier on its own and
//     reports the stage read on its "empty" mbarrier (no answer needed); the warps take turns at
//     waiting for all eight reports and refilling the stage (TMA of the chunk n_stages ahead);
//     the last warp to finish a segment combines the eight states and writes the result, while
//     the others are already in the next segment.  q of a cache rides along with the first tile of its segment (one more
//     bulk copy onto the same mbarrier);
//   * segments of a cache that spans several CTAs are combined by the warp that finishes last
//     (ticket), in CTA order, reading the partial results from L2;
//   * exponentials are taken in base 2 (scores pre-multiplied by log2 e, ex2.approx: relative
//     error 2^-22).
// Rows past a slot's position inside the last tile are masked (score -inf, weight 0); the caches are
// zero-initialised and only ever hold finite values, so the masked V rows contribute exactly 0.
// Waits on the copies are bounded (error bit 16 in *err; the CTA stops and drains).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "forward_kernels.cuh"
#include "gemm_tc.cuh"
#include "round_kernel.cuh"

namespace tabed {

constexpr int kAtcThreads = 256;
constexpr int kAtcWarps = kAtcThreads / 32;
constexpr int kAtcSplit = 128;               // positions per chunk = rows of a TMA tile
constexpr int kAtcHd = 64;                   // head size served by this kernel
constexpr int kAtcTile = kAtcSplit * kAtcHd * 2;   // bytes of one K (or V) tile
constexpr int kAtcMaxStages = 8;
constexpr int kAtcMaxCtas = 1024;
constexpr int kAtcMaxSlots = 512;
constexpr unsigned kAtcMaxDynSmem = 220u * 1024u;   // dynamic shared memory of a CTA that has the SM to itself (static: ~3 KB)

struct AttnTcArgs {
  const float* qkv;                          // [n_slots][qkv_w] rotated q (k, v already in the caches)
  const SlotDesc* slots;
  int n_slots, H, Hkv, layer, L, cap, qkv_w;
  float *part_o, *part_ml;                   // [n_slots][H][max_splits][hd], [..][2] segment partials
  int max_splits;
  int* tickets;                              // [n_slots][Hkv], zero on entry and on exit
  float* out;                                // [n_slots][H][hd]; unused when act_out is given
  unsigned char* act_out;                    // or null: the output as the bf16 B operand of the next projection
  int act_npad;                              //   (core-matrix layout of k_gemm_tc for act_npad slots, K = H * hd)
  float scale;
  int* err;
  int n_stages;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// x = hi + lo with hi, lo bf16 (lo the rounded remainder); returns them packed for two values
__device__ __forceinline__ void split_bf16x2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const float h0 = round_bf16(x0), h1 = round_bf16(x1);
  hi = pack_bf16(h0, h1);
  lo = pack_bf16(x0 - h0, x1 - h1);
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kAtcThreads, 2)
k_attn_tc_bf16(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, const AttnTcArgs A) {
  constexpr int HD = kAtcHd, NW = kAtcWarps, SPLIT = kAtcSplit;
  constexpr unsigned FULL = 0xffffffffu;
  const int H = A.H, Hkv = A.Hkv, grp = H / Hkv, NC = gridDim.x, cta = blockIdx.x, n_slots = A.n_slots;
  const int n_stages = A.n_stages;
  const SlotDesc* __restrict__ slots = A.slots;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, g = lane >> 2, t4 = lane & 3;
  pdl_trigger();
  extern __shared__ unsigned char atc_raw[];
  unsigned char* stage0 = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(atc_raw) + 1023) & ~(uintptr_t)1023);
  float* sq = reinterpret_cast<float*>(stage0 + (size_t)n_stages * 2 * kAtcTile);   // [n_stages][grp][HD] q beside its stage
  // The warps' states of a segment go through a ring of n_stages + 1 buffers: a warp can be n_stages chunks (hence
  // segments) ahead of the slowest one - the refill of a stage waits for all warps' reads, not for their segment
  // ends - and must not touch the buffer that warp's segment is still being combined from.
  const int n_segbuf = n_stages + 1;
  float* so = sq + (size_t)n_stages * grp * HD;                                     // [n_segbuf][NW][grp][HD] states of a segment
  float* sm = so + (size_t)n_segbuf * NW * grp * HD;                                // [n_segbuf][NW][grp] running maxima (base 2)
  float* sl = sm + n_segbuf * NW * grp;                                             // [n_segbuf][NW][grp] running sums
  __shared__ uint64_t full[kAtcMaxStages];
  __shared__ uint64_t empty[kAtcMaxStages];     // a stage's tiles have been read by all eight warps
  __shared__ int s_seg[kAtcMaxStages + 1];      // warps that have finished a segment (ring of n_stages + 1 segments)
  __shared__ int s_pref[kAtcMaxSlots + 1];
  __shared__ int s_start;
  if (tid == 0) {
    for (int i = 0; i < n_stages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], NW); }
    for (int i = 0; i <= n_stages; ++i) s_seg[i] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  pdl_wait();                                   // the slot table, q and the appended K, V come from the kernels before
  // chunks before every slot (prefix sums), built by the whole CTA
  for (int i = tid; i < n_slots; i += kAtcThreads)
    s_pref[i + 1] = slots[i].active ? Hkv * ((slots[i].pos + SPLIT) / SPLIT) : 0;
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int base = 0; base < n_slots; base += 32) {
      int v = (base + lane < n_slots) ? s_pref[base + lane + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int n = __shfl_up_sync(FULL, v, o); if (lane >= o) v += n; }
      if (base + lane < n_slots) s_pref[base + lane + 1] = carry + v;
      carry += __shfl_sync(FULL, v, 31);
    }
    if (lane == 0) s_pref[0] = 0;
  }
  __syncthreads();
  const int T = s_pref[n_slots];
  const int g_lo = (int)((long long)cta * T / NC), g_hi = (int)((long long)(cta + 1) * T / NC);
  for (int i = tid; i < n_slots; i += kAtcThreads)
    if (s_pref[i] <= g_lo && g_lo < s_pref[i + 1]) s_start = i;
  struct Walk { int s, gk, split, nsplit, row, pos; };
  auto advance = [&](Walk& w) {                      // to the next chunk in (slot, head, position) order
    w.split++;
    if (w.split == w.nsplit) {
      w.split = 0; w.gk++;
      if (w.gk == Hkv) {
        w.gk = 0;
        do { w.s++; } while (w.s < n_slots && !slots[w.s].active);
        if (w.s < n_slots) { w.row = slots[w.s].row; w.pos = slots[w.s].pos; }
        w.nsplit = (w.pos + SPLIT) / SPLIT;
      }
    }
  };
  auto seek = [&](int g, Walk& w) {                 // the (slot, head, split) of global chunk g < T
    int lo = 0, hi = n_slots;
    while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (s_pref[mid] <= g) lo = mid; else hi = mid; }
    w.s = lo; w.row = slots[lo].row; w.pos = slots[lo].pos;
    w.nsplit = (w.pos + SPLIT) / SPLIT;
    const int rem = g - s_pref[lo];
    w.gk = rem / w.nsplit; w.split = rem - w.gk * w.nsplit;
  };
  // one thread: the two TMA tiles of chunk `w` into stage `st`; q of the cache with the first chunk of a segment
  auto issue = [&](const Walk& w, int st, bool first) {
    const int y = ((w.row * A.L + A.layer) * Hkv + w.gk) * A.cap + w.split * SPLIT;
    const uint32_t dst = smem_u32(stage0 + (size_t)st * 2 * kAtcTile), bar = smem_u32(&full[st]);
    const bool with_q = first || w.split == 0;
    const unsigned qbytes = (unsigned)grp * HD * 4u;
    mbar_expect_tx(&full[st], 2u * kAtcTile + (with_q ? qbytes : 0u));
    tma_load_2d(dst, &tm_k, 0, y, bar);
    tma_load_2d(dst + kAtcTile, &tm_v, 0, y, bar);
    if (with_q) bulk_g2s(sq + (size_t)st * grp * HD, A.qkv + (size_t)w.s * A.qkv_w + (size_t)w.gk * grp * HD, qbytes, &full[st]);
  };
  // a lane's two output dims of (slot, head): fp32 rows, or straight into the next projection's operand blocks
  auto store_out = [&](int s, int head, float x0, float x1) {
    if (A.act_out) {
      const int k = head * HD + 2 * lane;          // column of the projection's input
      unsigned char* blk = A.act_out + (size_t)(k / kTcKC) * tc_block_bytes(A.act_npad);
      *reinterpret_cast<uint32_t*>(blk + ((size_t)((k % kTcKC) >> 3) * (A.act_npad >> 3) + (s >> 3)) * 128 + (s & 7) * 16 + (k & 7) * 2) =
          pack_bf16(x0, x1);
    } else {
      *reinterpret_cast<float2*>(A.out + ((size_t)s * H + head) * HD + 2 * lane) = make_float2(x0, x1);
    }
  };
  __syncthreads();
  // cur: the chunk a warp works on; ahead: the chunk n_stages later (the one that refills cur's stage)
  Walk cur{0, 0, 0, 1, 0, 0}, ahead{0, 0, 0, 1, 0, 0};
  if (g_lo < g_hi) {
    const int rem = g_lo - s_pref[s_start];
    cur.s = s_start;
    cur.row = slots[s_start].row; cur.pos = slots[s_start].pos;
    cur.nsplit = (cur.pos + SPLIT) / SPLIT;
    cur.gk = rem / cur.nsplit;
    cur.split = rem - cur.gk * cur.nsplit;
    ahead = cur;
    for (int i = 0; i < n_stages; ++i) {
      if (tid == 0 && g_lo + i < g_hi) issue(ahead, i, i == 0);
      if (g_lo + i + 1 < g_hi) advance(ahead);
    }
  }
  // per-warp running state of the current segment.  The products are taken with the POSITIONS (scores) and the DIMS
  // (output) as the 16 rows of the A operand and the group's query heads as the 8 columns of B: a cache tile is then
  // covered by half as many mma as with the heads as rows (of which at most 8 of 16 would be used).
  //   scores^T [16 positions x 8 heads] = K [16 x 64] q^T [64 x 8]          (4 k-steps, q as bf16 head + remainder)
  //   out^T    [64 dims x 8 heads]     += V^T [64 x 16] P^T [16 x 8]        (4 m-tiles, P as bf16 head + remainder)
  // Lane (g, t) holds columns (heads) 2t, 2t+1 of rows g, g+8; the softmax weights change from accumulator layout
  // (positions as rows) to B-operand layout (positions as the summed index) with movmatrix.
  uint32_t qh[4][2], ql[4][2];                  // B fragments of q^T per k-step (column g = head g; zero beyond the group)
  float o[4][4];                                // out^T: m-tile j = dims 16j .. 16j+15
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.0f, 0.0f};      // heads 2t, 2t+1; maxima in base-2 units
  int seg_first_split = 0, st = 0, seg_buf = 0;
  unsigned phase = 0;
  const float scale2 = A.scale * 1.4426950408889634f;
  const int r8 = lane & 7, ti = lane >> 3;
#pragma unroll 1
  for (int gi = g_lo; gi < g_hi; ++gi) {
    const int split = cur.split, nsplit = cur.nsplit;
    const int cnt = min(SPLIT, cur.pos + 1 - split * SPLIT);
    const bool have_next = gi + 1 < g_hi;
    const bool seg_start = (gi == g_lo) || split == 0;
    const bool seg_end = !have_next || split == nsplit - 1;
    {
      // every warp waits for the tiles on its own (also a warp without positions in this chunk: the
      // parity test is only valid for a warp that has seen every earlier phase complete)
      unsigned spins = 0;
      while (!mbar_try_wait(&full[st], phase)) {
        if (++spins > (1u << 20)) { if (lane == 0) atomicOr(A.err, 16); break; }     // reported; results are void
        if (spins > 4096) __nanosleep(64);
      }
    }
    if (seg_start) {
      seg_first_split = split;
      m_run[0] = m_run[1] = -INFINITY; l_run[0] = l_run[1] = 0.0f;
#pragma unroll
      for (int j = 0; j < 4; ++j) { o[j][0] = o[j][1] = o[j][2] = o[j][3] = 0.0f; }
      const float* qrow = sq + ((size_t)st * grp + g) * HD;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        float2 a = make_float2(0.0f, 0.0f), b = make_float2(0.0f, 0.0f);
        if (g < grp) {
          a = *reinterpret_cast<const float2*>(qrow + kk * 16 + 2 * t4);
          b = *reinterpret_cast<const float2*>(qrow + kk * 16 + 8 + 2 * t4);
        }
        split_bf16x2(a.x, a.y, qh[kk][0], ql[kk][0]);
        split_bf16x2(b.x, b.y, qh[kk][1], ql[kk][1]);
      }
    }
    if (warp * 16 < cnt) {
      const uint32_t kst = smem_u32(stage0 + (size_t)st * 2 * kAtcTile), vst = kst + kAtcTile;
      // scores of the warp's 16 positions for all heads of the group; four accumulators (q's head / remainder,
      // even / odd k-step) keep the dependent chains two mma long
      float sc[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) sc[j][0] = sc[j][1] = sc[j][2] = sc[j][3] = 0.0f;
      const uint32_t krow = kst + (uint32_t)(warp * 16 + (ti & 1) * 8 + r8) * 128u;
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        uint32_t ka[4];
        ldsm_x4(ka, krow + (uint32_t)(((2 * kk + (ti >> 1)) ^ r8) << 4));
        mma_bf16(sc[kk & 1], ka, qh[kk]);
        mma_bf16(sc[2 + (kk & 1)], ka, ql[kk]);
      }
      // softmax over the 16 positions, base 2: entries 0, 1 belong to position g, entries 2, 3 to position g + 8
      float sv[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        sv[e] = ((sc[0][e] + sc[1][e]) + (sc[2][e] + sc[3][e])) * scale2;
        if (cnt < SPLIT && warp * 16 + (e >> 1) * 8 + g >= cnt) sv[e] = -INFINITY;
      }
      float mx0 = fmaxf(sv[0], sv[2]), mx1 = fmaxf(sv[1], sv[3]);
#pragma unroll
      for (int ofs = 4; ofs < 32; ofs <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(FULL, mx0, ofs));
        mx1 = fmaxf(mx1, __shfl_xor_sync(FULL, mx1, ofs));
      }
      if (__any_sync(FULL, mx0 > m_run[0] || mx1 > m_run[1])) {      // a running maximum moves: rescale what has been gathered
        const float n0 = fmaxf(m_run[0], mx0), n1 = fmaxf(m_run[1], mx1);
        const float f0 = ex2_approx(m_run[0] - n0), f1 = ex2_approx(m_run[1] - n1);
        l_run[0] *= f0; l_run[1] *= f1;
#pragma unroll
        for (int j = 0; j < 4; ++j) { o[j][0] *= f0; o[j][2] *= f0; o[j][1] *= f1; o[j][3] *= f1; }
        m_run[0] = n0; m_run[1] = n1;
      }
      float pw[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { pw[e] = ex2_approx(sv[e] - m_run[e & 1]); l_run[e & 1] += pw[e]; }
      uint32_t ph[2], pl[2], h01, l01, h23, l23;
      split_bf16x2(pw[0], pw[1], h01, l01);
      split_bf16x2(pw[2], pw[3], h23, l23);
      ph[0] = movmatrix_trans(h01); ph[1] = movmatrix_trans(h23);
      pl[0] = movmatrix_trans(l01); pl[1] = movmatrix_trans(l23);
      // out^T += V^T P^T: the V tile transposed on load (rows = dims), the 16 positions are the summed index
      const uint32_t vrow = vst + (uint32_t)(warp * 16 + (ti >> 1) * 8 + r8) * 128u;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint32_t va[4];
        ldsm_x4_trans(va, vrow + (uint32_t)(((2 * j + (ti & 1)) ^ r8) << 4));
        mma_bf16(o[j], va, ph);
        mma_bf16(o[j], va, pl);
      }
    }
    // (the mma above have consumed every ldmatrix result)
    // every warp reports the stage read (no answer needed); the warps take turns at waiting for all eight
    // reports and refilling the stage with the chunk n_stages ahead
    __syncwarp();
    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&empty[st])) : "memory");
    if (((gi - g_lo) & (NW - 1)) == warp && gi + n_stages < g_hi) {
      seek(gi + n_stages, ahead);
      if (lane == 0) {
        unsigned spins = 0;
        while (!mbar_try_wait(&empty[st], phase)) {
          if (++spins > (1u << 20)) { atomicOr(A.err, 16); break; }      // reported; the round's results are void
          if (spins > 4096) __nanosleep(64);
        }
        issue(ahead, st, false);
      }
      __syncwarp();
    }
    if (++st == n_stages) { st = 0; phase ^= 1u; }
    if (seg_end) {
      // this warp's state -> shared memory; the last warp to get here combines the eight states
      float l_tot[2] = {l_run[0], l_run[1]};
#pragma unroll
      for (int ofs = 4; ofs < 32; ofs <<= 1) {
        l_tot[0] += __shfl_xor_sync(FULL, l_tot[0], ofs);
        l_tot[1] += __shfl_xor_sync(FULL, l_tot[1], ofs);
      }
      float* so_b = so + (size_t)seg_buf * NW * grp * HD;
      float* sm_b = sm + seg_buf * NW * grp;
      float* sl_b = sl + seg_buf * NW * grp;
#pragma unroll
      for (int e = 0; e < 2; ++e) {
        const int head = 2 * t4 + e;
        if (head < grp) {
          float* dst = so_b + ((size_t)warp * grp + head) * HD + g;
#pragma unroll
          for (int j = 0; j < 4; ++j) { dst[16 * j] = o[j][e]; dst[16 * j + 8] = o[j][2 + e]; }
          if (g == 0) { sm_b[warp * grp + head] = m_run[e]; sl_b[warp * grp + head] = l_tot[e]; }
        }
      }
      __syncwarp();
      int last = 0;
      if (lane == 0) {
        __threadfence_block();
        last = atomicAdd(&s_seg[seg_buf], 1) == NW - 1;
        if (last) { s_seg[seg_buf] = 0; __threadfence_block(); }
      }
      last = __shfl_sync(FULL, last, 0);
      if (last) {
        const int s = cur.s, gk = cur.gk;
        const bool whole = seg_first_split == 0 && split == nsplit - 1;
        const int g0 = gi - split;                 // first chunk of this cache
        int n_c = 0, c_a = 0;
        if (!whole) {
          c_a = (int)((((long long)g0 + 1) * NC - 1) / T);
          n_c = (int)((((long long)g0 + nsplit) * NC - 1) / T) - c_a + 1;
        }
        // first split of CTA (c_a + j)'s segment of this cache, or -1 when that CTA has no chunk at all
        auto seg_of = [&](int j) {
          const int lo_c = (int)((long long)(c_a + j) * T / NC), hi_c = (int)((long long)(c_a + j + 1) * T / NC);
          return (lo_c < hi_c) ? max(lo_c, g0) - g0 : -1;
        };
#pragma unroll 1
        for (int t = 0; t < grp; ++t) {
          float M = -INFINITY;
#pragma unroll
          for (int w = 0; w < NW; ++w) M = fmaxf(M, sm_b[w * grp + t]);
          float2 v = make_float2(0.0f, 0.0f);
          float l = 0.0f;
#pragma unroll
          for (int w = 0; w < NW; ++w) {
            const float f = ex2_approx(sm_b[w * grp + t] - M);      // 0 for a warp that saw no position
            const float2 x = *reinterpret_cast<const float2*>(so_b + ((size_t)w * grp + t) * HD + 2 * lane);
            v.x = fmaf(f, x.x, v.x); v.y = fmaf(f, x.y, v.y);
            l = fmaf(f, sl_b[w * grp + t], l);
          }
          const int head = gk * grp + t;
          if (whole) {
            store_out(s, head, v.x / l, v.y / l);
          } else {
            const size_t pi = ((size_t)s * H + head) * A.max_splits + seg_first_split;
            *reinterpret_cast<float2*>(A.part_o + pi * HD + 2 * lane) = v;
            if (lane == 0) { A.part_ml[pi * 2] = M; A.part_ml[pi * 2 + 1] = l; }
          }
        }
        if (!whole) {
          __syncwarp();
          int fin = 0;
          if (lane == 0) {
            __threadfence();                       // the warp's partial results before the ticket
            int n_seg = 0;
            for (int j = 0; j < n_c; ++j) n_seg += seg_of(j) >= 0;
            fin = atomicAdd(A.tickets + s * Hkv + gk, 1) == n_seg - 1;
            if (fin) __threadfence();
          }
          fin = __shfl_sync(FULL, fin, 0);
          if (fin) {                               // every segment of the cache is in L2: combine them in CTA order
#pragma unroll 1
            for (int t = 0; t < grp; ++t) {
              const int head = gk * grp + t;
              const size_t base = ((size_t)s * H + head) * A.max_splits;
              float M = -INFINITY;
              for (int j = 0; j < n_c; ++j) { const int f0 = seg_of(j); if (f0 >= 0) M = fmaxf(M, __ldcg(A.part_ml + (base + f0) * 2)); }
              float2 num = make_float2(0.0f, 0.0f);
              float den = 0.0f;
              for (int j = 0; j < n_c; ++j) {
                const int f0 = seg_of(j);
                if (f0 < 0) continue;
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(A.part_ml + (base + f0) * 2));
                const float f = ex2_approx(ml.x - M);
                const float2 x = __ldcg(reinterpret_cast<const float2*>(A.part_o + (base + f0) * HD + 2 * lane));
                num.x = fmaf(f, x.x, num.x); num.y = fmaf(f, x.y, num.y);
                den = fmaf(f, ml.y, den);
              }
              store_out(s, head, num.x / den, num.y / den);
            }
            if (lane == 0) A.tickets[s * Hkv + gk] = 0;
          }
        }
      }
      if (++seg_buf == n_segbuf) seg_buf = 0;
    }
    if (have_next) advance(cur);
  }
}

}  // namespace tabed
