// Persistent kernel for one whole drafting round (Algorithm 1 steps 4-8): gamma batched
// shared-weight decoder steps, each followed by softmax + weighted-average ensemble + draw, in ONE
// cooperative launch with one CTA per SM.
//
// Why one kernel: with m <= 4 drafting inputs a decoder step moves ~125-630 MB of weights through
// dozens of strictly dependent phases; as separate launches every phase pays a launch plus a cold
// DRAM round trip.  Here
//   * the weights never stop streaming: every CTA owns a fixed share of the weight tiles of every
//     phase (its unit list is built once, in shared memory), and a ring of shared-memory slots is
//     kept full by bulk asynchronous copies (cp.async.bulk + mbarrier) several phases ahead of the
//     arithmetic, so HBM stays busy across the phase boundaries;
//   * the weights are read from a private copy laid out for this kernel at set-up: every unit (16
//     output rows x kchunk input columns, rows padded to a bank-conflict-free shared-memory pitch)
//     is one contiguous block, hence ONE bulk copy;
//   * there is NO grid barrier.  Every activation that crosses CTAs travels as an 8-byte word
//     {value, epoch} written with one 64-bit store; the epoch names the launch, the step and the
//     phase that produced it, so a consumer polls the data itself and starts as soon as ITS inputs
//     have arrived (one L2 round trip per phase instead of an arrive/spin pair, and no CTA waits
//     for producers it does not read).  A phase is: stage the (tiny) activations by polling their
//     words -> tensor-core products of the weight tiles already sitting in shared memory -> flagged
//     results back to L2.  5 phases per layer (QKV, attention, O, gate/up, down).  A 16-row tile
//     always takes its whole input dimension on ONE CTA (long rows as sub-units whose products
//     accumulate in registers), so no projection leaves split-K partial sums behind; residual adds
//     ride in the epilogues and every consumer computes the RMSNorm sum of squares itself from the
//     words it stages (warp per input row, fixed order: deterministic);
//   * a poll re-requests all words still missing together; after two empty rounds one lane per
//     warp keeps polling with a back-off while the others idle, so that long waits do not flood L2
//     - all 32 lanes of a warp therefore enter the staging helpers together;
//   * four warp groups work on four units at a time (mma.sync m16n8k16, bf16 x bf16 -> fp32:
//     16 weight rows x up to 8 slots).  The contraction is HBM-bound (<= 8 flop per weight byte);
//     the tensor pipe only keeps the ALUs off the critical path;
//   * attention: a CTA walks a contiguous range of cache chunks; head size 64 runs on mma
//     fragments loaded straight from global memory; the partial results of a cache are put
//     together by the next phase's staging (a per-step table says how many partials each
//     (slot, head) has);
//   * all cross-CTA data is read with relaxed gpu-scope loads (L2): L1 is not coherent across SMs;
//   * loops are deliberately not unrolled except the few hot ones: every phase runs its code once,
//     so unrolling buys nothing and only inflates the instruction footprint.
//
// Rows: up to 4 rows feed both pending tokens of a fully accepted block in the first step's weight pass
// (2 R <= 8 slots); with 5 - 8 rows the first of the two gets a pass of its own before step 0 (all layers,
// no LM head, only the rows that have two pending tokens are active), so a pass never has more than 8 slots.
//
// Waits are bounded: a flagged word or a copy that does not arrive within the spin limit sets an
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
constexpr int kWG = 4;                   // warp groups (each works on its own unit)
constexpr int kGW = kPW / kWG;           // warps per group
constexpr int kPSlots = 8;               // slots (row, position) per step: one mma n-tile
constexpr int kPRing = 16;               // upper bound of ring slots
constexpr int kPPer = kChunk / kPT;      // vocabulary elements per thread and chunk (4)
constexpr int kPMaxD = 2048;             // d_model bound
constexpr int kTraceRec = 8;             // words per record of the phase timeline
constexpr int kPMaxL = 64;               // layers (their pointer table lives in shared memory)
constexpr int kPMaxHeads = 64;           // query heads
constexpr int kMaxUnits = 1024;          // units of one CTA in one decoder step (config 3 needs 168)
constexpr int kMaxPhase = 4 * kPMaxL + 1;

enum { KIND_QKV = 0, KIND_O = 1, KIND_GU = 2, KIND_DN = 3, KIND_LM = 4 };
enum { PERR_BARRIER = 8, PERR_COPY = 16, PERR_KV = 4 };

struct LayerW { const __nv_bfloat16 *wq, *wk, *wv, *wo, *wg, *wu, *wd, *n1, *n2; };

// A phase's weight matrix is cut into tiles of 16 output rows; a tile is nsub units of kchunk input
// columns each (nsub in {1, 2} or a multiple of 4).  unit u -> tile = u / nsub, sub = u % nsub.
struct PhaseGeom { int n_tiles, nsub, kchunk, n_units; };

struct RoundArgs {
  // drafter
  const LayerW* layers;
  const __nv_bfloat16 *embed, *final_norm;
  const float *rope_cos, *rope_sin;
  int L, d, F, H, Hkv, hd, V, cap, qkv_w;
  float eps, attn_scale;
  PhaseGeom geom[5];
  const unsigned char* packed;          // weights re-laid out unit by unit (k_pack_units)
  unsigned long long pack_off[5];       // byte offset of a kind's units inside a layer block (LM: absolute)
  unsigned long long pack_layer_stride;
  int slot_bytes, n_ring, act_bytes, act_slots, split_len;
  // round
  int R, B, m, G, greedy;
  const int* kv_len;                    // [R] committed lengths (constant during the round)
  const int* pending;                   // [B][3]
  __nv_bfloat16 *kc, *vc;               // [R][L][Hkv][cap][hd]
  // activations exchanged through L2 as {value, epoch} pairs (one 8-byte store, polled by the consumer)
  uint2 *xa, *x1;                       // [8][d] residual entering a layer / after its attention block
  uint2* qkv;                           // [8][qkv_w]
  uint2* mid;                           // [8][F/2] two bf16 values of the gated product per pair
  uint2 *part_o, *part_ml;              // attention partials [8][H][max_splits][hd], [..][2] (max, sum)
  int max_splits;
  unsigned epoch0;                      // the launch's first epoch; phase p of pass i stamps epoch0 + i * (5 L + 8) + p + 1
  int prepass;                          // more than kPSlots / 2 rows: a fully accepted block's first pending token is fed in a
                                        // pass of its own (all layers, no LM head) before step 0, instead of as R more slots
  // ensemble
  float* logits_own;                    // [G][R][V]
  const float* logits_override;         // or null
  const float* w;                       // [B][m]
  const float* u;                       // [B][G]
  float *qk, *q;                        // [B][G][m][V], [B][G][V]
  uint2 *rowmax, *rowmax2;              // [CTAs][8] every CTA's maxima of the logit rows (LM head; the logits of a replay)
  uint2* rowsum;                        // [CTAs][8][2] every CTA's integer exp sums, low and high word
  uint2* chunk_mass;                    // [B][n_chunks][2] mass of a chunk of q, low and high word (greedy: best value, its index)
  int n_chunks;
  int *tokens, *out_tokens;             // [B][G]
  // diagnostics
  int* err;
  unsigned long long* trace;            // optional [G][trace_stride][kTraceRec] phase timeline
  int trace_stride, trace_cta;          // the CTA that records
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
// transposes an 8 x 8 matrix of 16-bit elements held one row per quad (lane (g, t): row g, columns 2t, 2t+1)
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
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
// Flagged words: an aligned 8-byte {value, epoch} pair is written by ONE store and read by one load, so a
// reader sees either the old pair or the new one; a 16-byte load returns two such pairs.
__device__ __forceinline__ void ll_store(uint2* p, uint32_t value, uint32_t epoch) {
  asm volatile("st.relaxed.gpu.global.v2.u32 [%0], {%1, %2};" ::"l"(p), "r"(value), "r"(epoch) : "memory");
}
__device__ __forceinline__ uint2 ll_load1(const uint2* p) {
  uint2 v;
  asm volatile("ld.relaxed.gpu.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ uint4 ll_load2(const uint2* p) {           // p 16-byte aligned: pairs p[0], p[1]
  uint4 v;
  asm volatile("ld.relaxed.gpu.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
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

__device__ __forceinline__ float4 bf16x4_to_float4(uint2 v) {
  return make_float4(__uint_as_float(v.x << 16), __uint_as_float(v.x & 0xFFFF0000u),
                     __uint_as_float(v.y << 16), __uint_as_float(v.y & 0xFFFF0000u));
}

// ------------------------------------------------------------------------------------------------
// per-CTA state
// ------------------------------------------------------------------------------------------------
struct PSlot { int row, pos, active, tok; };

struct PShared {
  uint64_t full[kPRing];
  LayerW layers[kPMaxL];
  uint32_t ulist[kMaxUnits];            // this CTA's units of one decoder step, in consumption order
  uint16_t pstart[kMaxPhase + 1];       // first entry of every phase in ulist
  float sc[kMaxGroup][4];               // scores of the positions produced in this very phase (at most 2)
  alignas(16) float q[kMaxGroup][128];
  float kf[2][128], vf[2][128];
  float red[kPW][kPSlots];
  float red2[kPW][kPSlots];
  unsigned long long red64[kPW];
  unsigned long long cm[kPT];
  float bestv[kPW]; int besti[kPW];
  float scale[kPSlots];
  uint32_t lmmax[kPSlots];
  float mix_mx[kMaxInputs], mix_sn[kMaxInputs], mix_w[kMaxInputs];
  float m_[kMaxGroup], l_[kMaxGroup];
  PSlot slot[kPSlots];
  int lm_src[kPSlots];
  int att[8];                           // attention geometry of the step: T, g_lo, g_hi, then this CTA's first chunk (s, gk, split, nsplit, g0)
  int pair_base[kPSlots], pair_ns[kPSlots];   // per slot: chunks before its first pair, chunks per pair (0: inactive)
  unsigned char nseg[kPSlots][kPMaxHeads];    // per (slot, head): partial attention results of the step
  int tok[kPSlots];
  float rowmax_f[kPSlots];
  unsigned long long row_part[kPSlots];
  int dead, flag, result, chunk;
  unsigned long long thr;
};

// a unit of the list: kind (3 bits), layer (7), sub-unit of its tile (6), tile (16) - no division where it is used
__device__ __forceinline__ uint32_t unit_pack(int kind, int layer, int tile, int sub) {
  return (uint32_t)kind | ((uint32_t)layer << 3) | ((uint32_t)sub << 10) | ((uint32_t)tile << 16);
}
__device__ __forceinline__ int unit_sub(uint32_t e) { return (int)((e >> 10) & 63u); }
__device__ __forceinline__ int unit_tile(uint32_t e) { return (int)(e >> 16); }

// Issue the bulk copy of unit number k (counted over the whole round) into its ring slot (one thread).
// The stream of units is [the list without its LM-head units, if the round has the extra pass] then the whole list per step.
__device__ __forceinline__ void issue_unit(const RoundArgs& A, PShared& S, unsigned char* ring, unsigned k, unsigned per_step, unsigned pre_units) {
  const uint32_t e = S.ulist[k < pre_units ? k : (k - pre_units) % per_step];
  const int kind = e & 7, layer = (e >> 3) & 127, u = unit_tile(e) * A.geom[kind].nsub + unit_sub(e);
  const unsigned bytes = 16u * ((unsigned)A.geom[kind].kchunk * 2u + 16u);
  const unsigned char* src = A.packed + A.pack_off[kind] + (size_t)u * bytes +
                             (kind == KIND_LM ? 0ull : (unsigned long long)layer * A.pack_layer_stride);
  const int slot = (int)(k % (unsigned)A.n_ring);
  mbar_expect_tx(&S.full[slot], bytes);
  bulk_g2s(ring + (size_t)slot * A.slot_bytes, src, bytes, &S.full[slot]);
}

// Re-lay one weight matrix (or the QKV / gate-up group) of one layer into units.  grid (n_units), block 256.
// Row r of unit (tile, sub): QKV rows are the concatenation wq | wk | wv; gate/up units hold 8 gate
// rows then the 8 matching up rows; LM-head rows beyond V are zero.
struct PackArgs {
  const __nv_bfloat16 *w0, *w1, *w2;    // source matrices [rows_i][K]
  int rows0, rows1, rows2, K, kind;
  PhaseGeom g;
  unsigned char* dst;                   // first unit of this (layer, kind)
};
__global__ void k_pack_units(const PackArgs P) {
  const int u = blockIdx.x;
  const int tile = u / P.g.nsub, sub = u - tile * P.g.nsub;
  const int pitch = P.g.kchunk * 2 + 16;
  unsigned char* unit = P.dst + (size_t)u * 16 * pitch;
  const int vec_per_row = pitch / 16;                      // 16-byte vectors per padded row
  for (int idx = threadIdx.x; idx < 16 * vec_per_row; idx += blockDim.x) {
    const int r = idx / vec_per_row, c16 = idx - r * vec_per_row;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (c16 * 8 < P.g.kchunk) {
      const __nv_bfloat16* base = nullptr;
      int row;
      if (P.kind == KIND_GU) { row = tile * 8 + (r & 7); base = (r < 8) ? P.w0 : P.w1; if (row >= P.rows0) base = nullptr; }
      else {
        row = tile * 16 + r;
        if (row < P.rows0) base = P.w0;
        else if (row < P.rows0 + P.rows1) { base = P.w1; row -= P.rows0; }
        else if (row < P.rows0 + P.rows1 + P.rows2) { base = P.w2; row -= P.rows0 + P.rows1; }
      }
      if (base) v = *reinterpret_cast<const uint4*>(base + (size_t)row * P.K + (size_t)sub * P.g.kchunk + c16 * 8);
    }
    *reinterpret_cast<uint4*>(unit + (size_t)r * pitch + (size_t)c16 * 16) = v;
  }
}

constexpr unsigned kSpinLimit = 1u << 21;

// Bounded wait for a ring slot.  Returns false on timeout.
__device__ __forceinline__ bool wait_full(PShared& S, int slot, unsigned parity, int* err) {
  unsigned spins = 0;
  while (!mbar_try_wait(&S.full[slot], parity)) {
    if (++spins > kSpinLimit) { atomicOr(err, PERR_COPY); return false; }
    if (spins > 4096) __nanosleep(64);
  }
  return true;
}

// Bounded polls of flagged words.  On a timeout the error bit is set and S.dead raised; the caller leaves
// after its next block-wide barrier.
__device__ __noinline__ void ll_timeout(PShared& S, int* err) {
  atomicOr(err, PERR_BARRIER);
  S.dead = 1;
}
__device__ __forceinline__ uint32_t ll_wait1(const uint2* p, uint32_t epoch, PShared& S, int* err) {
  uint2 v = ll_load1(p);
  unsigned spins = 0;
  while (v.y != epoch) {
    if (++spins > kSpinLimit) { ll_timeout(S, err); break; }
    if (spins > 256) __nanosleep(spins > 4096 ? 64 : 20);
    v = ll_load1(p);
  }
  return v.x;
}
// A long wait must not flood L2 with polls (75 000 threads would): after two rounds in which some lane of the warp
// still misses a word, ONE lane keeps polling one missing word, with growing pauses, while the others idle; then the
// whole warp looks again.  All 32 lanes call these helpers together (lanes without work pass n = 0 / null).
__device__ __forceinline__ void ll_backoff_wait1(const uint2* p, uint32_t epoch, unsigned& spins, PShared& S, int* err) {
  unsigned ns = 40;
  while (ll_load1(p).y != epoch) {
    if (++spins > kSpinLimit) { ll_timeout(S, err); break; }
    __nanosleep(ns);
    if (ns < 400) ns += 40;
  }
}
// Several 16-byte loads in flight (the word pairs at addr(j), j < n); every round re-requests ALL the ones that do
// not carry the epoch yet, together, so that a wait costs one more trip to L2 however many words were missing.
template <int N, typename AddrFn>
__device__ __forceinline__ void ll_poll(AddrFn addr, int n, uint32_t epoch, uint4 (&v)[N], PShared& S, int* err) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int j = 0; j < N; ++j) {
    const uint2* pj = j < n ? addr(j) : nullptr;              // (a null address: nothing to wait for)
    v[j] = pj ? ll_load2(pj) : make_uint4(0u, epoch, 0u, epoch);
  }
  unsigned spins = 0, rounds = 0;
  while (true) {
    const uint2* pmiss = nullptr;                             // one word this lane still misses
#pragma unroll
    for (int j = 0; j < N; ++j)
      if (j < n && !pmiss && (v[j].y != epoch || v[j].w != epoch)) pmiss = addr(j) + (v[j].y != epoch ? 0 : 1);
    const unsigned who = __ballot_sync(0xffffffffu, pmiss != nullptr);
    if (!who) break;
    if (++spins > kSpinLimit) { ll_timeout(S, err); break; }
    if (++rounds > 2) {
      if (lane == __ffs(who) - 1) ll_backoff_wait1(pmiss, epoch, spins, S, err);
      __syncwarp();
      if (S.dead) break;
    }
#pragma unroll
    for (int j = 0; j < N; ++j) if (j < n && (v[j].y != epoch || v[j].w != epoch)) v[j] = ll_load2(addr(j));
  }
}
__device__ __forceinline__ uint4 ll_wait2(const uint2* p, uint32_t epoch, PShared& S, int* err) {       // p null: lane without a word
  uint4 v[1] = {make_uint4(0u, epoch, 0u, epoch)};
  ll_poll<1>([&](int) { return p; }, p ? 1 : 0, epoch, v, S, err);
  return v[0];
}
// two single words in flight (either may be null)
__device__ __forceinline__ void ll_wait1x2(const uint2* p0, const uint2* p1, uint32_t epoch, uint32_t& x0, uint32_t& x1, PShared& S, int* err) {
  const int lane = threadIdx.x & 31;
  uint2 a = p0 ? ll_load1(p0) : make_uint2(0u, epoch), b = p1 ? ll_load1(p1) : make_uint2(0u, epoch);
  unsigned spins = 0, rounds = 0;
  while (true) {
    const bool ra = a.y != epoch, rb = b.y != epoch;
    const unsigned who = __ballot_sync(0xffffffffu, ra || rb);
    if (!who) break;
    if (++spins > kSpinLimit) { ll_timeout(S, err); break; }
    if (++rounds > 2) {
      if (lane == __ffs(who) - 1) ll_backoff_wait1(ra ? p0 : p1, epoch, spins, S, err);
      __syncwarp();
      if (S.dead) break;
    }
    if (ra) a = ll_load1(p0);
    if (rb) b = ll_load1(p1);
  }
  x0 = a.x; x1 = b.x;
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
template <bool TRACE>
__global__ void __launch_bounds__(kPT, 1) k_draft_round(const RoundArgs A) {
  extern __shared__ __align__(128) unsigned char dyn_smem[];
  __shared__ PShared S;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wgrp = warp / kGW, wl = warp % kGW;          // warp group and warp within the group
  const int cta = blockIdx.x, NC = gridDim.x;
  unsigned char* ring = dyn_smem;
  unsigned char* U = dyn_smem + (size_t)A.n_ring * A.slot_bytes;
  __nv_bfloat16* act = reinterpret_cast<__nv_bfloat16*>(U);               // [areas][act_slots][apitch]
  float* cpart = reinterpret_cast<float*>(U + A.act_bytes);               // [2][kPW][128]
  float* s_o = reinterpret_cast<float*>(U);                               // attention: [kPW][grp*hd]
  const int kvd = A.Hkv * A.hd, grp = A.H / A.Hkv, half = A.hd >> 1;
  const int R = A.R, B = A.B, m = A.m, G = A.G, V = A.V, d = A.d;
  const int n_phase = 4 * A.L + 1;

  // ---- set-up -----------------------------------------------------------------------------------
  if (tid == 0) {
#pragma unroll 1
    for (int s = 0; s < A.n_ring; ++s) mbar_init(&S.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    S.dead = 0;
  }
#pragma unroll 1
  for (int i = tid; i < A.L * (int)(sizeof(LayerW) / sizeof(void*)); i += kPT)
    reinterpret_cast<const void**>(S.layers)[i] = reinterpret_cast<const void* const*>(A.layers)[i];
  // unit list of one decoder step: tiles of phase p are dealt round-robin over the CTAs, starting
  // where phase p-1 stopped, so that every CTA streams about the same number of bytes
#pragma unroll 1
  for (int p = tid; p <= n_phase; p += kPT) {
    int cnt = 0;
    if (p < n_phase) {
      const int kind = (p == n_phase - 1) ? KIND_LM : (p & 3);
      int off = 0;                                     // tiles dealt before this phase, modulo NC
#pragma unroll 1
      for (int q2 = 0; q2 < p; ++q2) off = (off + A.geom[(q2 & 3)].n_tiles) % NC;
      int first = cta - off;
      if (first < 0) first += NC;
      const int nt = A.geom[kind].n_tiles;
      cnt = (first < nt) ? ((nt - 1 - first) / NC + 1) * A.geom[kind].nsub : 0;
    }
    S.pstart[p] = (uint16_t)cnt;                       // counts first, offsets after the scan below
  }
  __syncthreads();
  if (tid == 0) {
    int run = 0;
#pragma unroll 1
    for (int p = 0; p <= n_phase; ++p) { const int c2 = S.pstart[p]; S.pstart[p] = (uint16_t)run; run += c2; }
  }
  __syncthreads();
#pragma unroll 1
  for (int p = tid; p < n_phase; p += kPT) {
    const int kind = (p == n_phase - 1) ? KIND_LM : (p & 3);
    int off = 0;
#pragma unroll 1
    for (int q2 = 0; q2 < p; ++q2) off = (off + A.geom[(q2 & 3)].n_tiles) % NC;
    int first = cta - off;
    if (first < 0) first += NC;
    int n = S.pstart[p];
    const int nsub = A.geom[kind].nsub;
#pragma unroll 1
    for (int t = first; t < A.geom[kind].n_tiles; t += NC)
#pragma unroll 1
      for (int sb = 0; sb < nsub; ++sb) S.ulist[n++] = unit_pack(kind, p >> 2, t, sb);
  }
  __syncthreads();
  const unsigned per_step = S.pstart[n_phase];
  // the extra pass: only in a round in which some request has two pending tokens (the same answer in every CTA)
  int pre = 0;
  if (A.prepass) {
#pragma unroll 1
    for (int b = 0; b < B; ++b) if (A.pending[b * 3] == 2) pre = 1;
  }
  const unsigned pre_units = pre ? S.pstart[n_phase - 1] : 0u;     // its units: every phase but the LM head
  const unsigned total_units = pre_units + per_step * (unsigned)G;
  if (tid == 0) {
#pragma unroll 1
    for (unsigned k = 0; k < (unsigned)A.n_ring && k < total_units; ++k) issue_unit(A, S, ring, k, per_step, pre_units);
  }
  bool alive = true;
  const unsigned EPS = 5u * (unsigned)A.L + 8u;          // epochs per decoder step
  unsigned cons_done = 0;                                // units consumed so far (for the drain)

  // phase timeline (CTA 0, thread 0): per grid barrier one record of kTraceRec words:
  // [0] nanosecond timer after the barrier, [1..6] clock cycles spent since the previous barrier in
  // staging activations, waiting for weight tiles, mma+partials, issuing copies + epilogue (for
  // attention: its four sections in slots 1-4), everything else, and in the barrier itself
  const bool tr_on = TRACE && A.trace != nullptr && cta == (A.trace_cta < NC ? A.trace_cta : 0) && tid == 0;
  long long t_sec[6] = {0, 0, 0, 0, 0, 0};
  long long t_mark = 0;
#define TSEC(k)                                       \
  do {                                                \
    if (TRACE && tr_on) {                             \
      const long long t_now = clock64();              \
      t_sec[k] += t_now - t_mark;                     \
      t_mark = t_now;                                 \
    }                                                 \
  } while (0)
  // End of a phase: nothing is waited for here (the next phase polls the words it needs); the timeline gets
  // its record, and a CTA that has seen a wait run out leaves.
#define PHASE_END()                                                        \
  do {                                                                     \
    TSEC(4);                                                               \
    if (TRACE && tr_on && step >= 0 && trace_n < A.trace_stride) {         \
      unsigned long long* rec = A.trace + ((size_t)(step < 0 ? 0 : step) * A.trace_stride + trace_n++) * kTraceRec; \
      rec[0] = global_timer();                                             \
      for (int k = 0; k < 6; ++k) { rec[1 + k] = (unsigned long long)t_sec[k]; t_sec[k] = 0; }     \
    }                                                                      \
    if (__syncthreads_or(S.dead)) { alive = false; goto drain; }           \
  } while (0)
  if (tr_on) t_mark = clock64();

#pragma unroll 1
  for (int it = 0; it < G + pre; ++it) {
    const int step = it - pre;                          // -1: the extra pass
    const unsigned ubase = step < 0 ? 0u : pre_units + (unsigned)step * per_step;    // first unit of this pass in the stream
    int trace_n = 0;
    // ---- slot table of the step ------------------------------------------------------------------
    int ns = R;
    if (step == 0 && !A.prepass) {
#pragma unroll 1
      for (int b = 0; b < B; ++b) if (A.pending[b * 3] == 2) ns = 2 * R;
    }
    if (tid < kPSlots) {
      PSlot sl{0, 0, 0, 0};
      if (tid < ns) {
        const int row = tid % R, b = row / m, second = tid >= R;
        const int* pend = A.pending + b * 3;
        sl.row = row;
        if (step < 0) {                                 // the first of two pending tokens, for the rows that have two
          sl.pos = A.kv_len[row];
          sl.tok = pend[1];
          sl.active = pend[0] == 2;
        } else if (step == 0 && A.prepass) {            // the last pending token
          sl.pos = A.kv_len[row] + pend[0] - 1;
          sl.tok = pend[pend[0]];
          sl.active = 1;
        } else if (step == 0) {
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
      S.lmmax[tid] = 0u;
      if (tid < R) {
        const int b = tid / m;
        S.lm_src[tid] = (step == 0 && !A.prepass && A.pending[b * 3] == 2) ? R + tid : tid;
      }
    }
    __syncthreads();
    if (tid == kPT - 32) {
      // (a thread of the last warp, off the path of the staging that follows; the result is first read at the end of
      // the QKV phase, several block-wide barriers later)
      // chunks of split_len positions of all (slot, KV head) caches in (slot, head, position) order; this CTA's
      // contiguous range of them and where it starts (the same for every layer of the step)
      const int sl = A.split_len;
      int T = 0;
#pragma unroll 1
      for (int s = 0; s < kPSlots; ++s) {
        const int nsp = (s < ns && S.slot[s].active) ? (S.slot[s].pos + sl) / sl : 0;
        S.pair_base[s] = T; S.pair_ns[s] = nsp;
        T += A.Hkv * nsp;
      }
      // (T <= 8 slots x 64 heads x 256 chunks, so c * T stays far below 2^31)
      const int lo = cta * T / NC, hi = (cta + 1) * T / NC;
      int s = 0, rem = lo, acc = 0, nsplit = 0;
      if (lo < hi) {
#pragma unroll 1
        for (; s < ns; ++s) {
          nsplit = S.slot[s].active ? (S.slot[s].pos + sl) / sl : 0;
          if (rem < A.Hkv * nsplit) break;
          rem -= A.Hkv * nsplit; acc += A.Hkv * nsplit;
        }
      }
      const int gk = nsplit ? rem / nsplit : 0;
      S.att[0] = T; S.att[1] = lo; S.att[2] = hi; S.att[3] = s; S.att[4] = gk; S.att[5] = nsplit ? rem - gk * nsplit : 0;
      S.att[6] = nsplit; S.att[7] = acc + gk * nsplit;
    }
    if (warp == kPW - 1) {
      // partial results every (slot, head) pair will have (first read by the O-projection staging): the last warp's lanes
      // share the pairs
      __syncwarp();
      const int T = S.att[0];
#pragma unroll 1
      for (int pr2 = lane; pr2 < kPSlots * A.Hkv; pr2 += 32) {
        const int s3 = pr2 / A.Hkv, gk3 = pr2 - s3 * A.Hkv;
        const int nsp = S.pair_ns[s3], g0 = S.pair_base[s3] + gk3 * nsp;
        const int cnt = nsp == 0 ? 0 : ((T >= NC) ? ((g0 + nsp) * NC - 1) / T - ((g0 + 1) * NC - 1) / T + 1 : nsp);
#pragma unroll 1
        for (int t3 = 0; t3 < grp; ++t3) S.nseg[s3][gk3 * grp + t3] = (unsigned char)cnt;
      }
    }

#pragma unroll 1
    for (int phase = 0; phase < (step < 0 ? n_phase - 1 : n_phase); ++phase) {
      const int kind = (phase == n_phase - 1) ? KIND_LM : (phase & 3);
      const int layer = phase >> 2;
      const LayerW& lw = S.layers[kind == KIND_LM ? 0 : layer];
      const PhaseGeom g = A.geom[kind];
      const int apitch = g.kchunk + 8;                       // bf16 elements
      const int area_elems = A.act_slots * apitch;           // one staging area: [act_slots][apitch]
      const int n_in = (kind == KIND_LM) ? R : ns;           // activation rows of the phase
      const bool norm_kind = kind == KIND_QKV || kind == KIND_GU || kind == KIND_LM;
      const unsigned ka = ubase + S.pstart[phase], kb = ubase + S.pstart[phase + 1];

      // epochs of the words this phase reads and writes
      const unsigned ep_base = A.epoch0 + (unsigned)it * EPS;
      const unsigned ep_prev_dn = ep_base + 5u * (unsigned)layer;                    // down projection of the layer before
      const unsigned ep_qkv = ep_base + 5u * (unsigned)layer + 1u, ep_att = ep_qkv + 1u, ep_o = ep_qkv + 2u, ep_gu = ep_qkv + 3u,
                     ep_dn = ep_qkv + 4u, ep_lm = ep_base + 5u * (unsigned)A.L + 1u;
      if (norm_kind && ka < kb) {
        // ---- stage RMSNorm(x) * gain as bf16, whole rows (these phases have kchunk == d) -----------
        // Warp w serves input row w % n_in; a row's warps walk its 16-byte pieces (two flagged words = two
        // elements) with every load in flight at once.  The sum of squares is taken per warp and the warps of a
        // row are added in warp order: the same bits in every CTA and in every run.
        const bool from_embed = kind == KIND_QKV && layer == 0;
        const uint2* xbuf = (kind == KIND_GU) ? A.x1 : A.xa;
        const unsigned ep_in = (kind == KIND_GU) ? ep_o : (kind == KIND_LM ? ep_base + 5u * (unsigned)A.L : ep_prev_dn);
        const __nv_bfloat16* gain = (kind == KIND_QKV) ? lw.n1 : (kind == KIND_GU ? lw.n2 : A.final_norm);
        const int s = warp % n_in, wi = warp / n_in, nw = (kPW - s + n_in - 1) / n_in;
        const int src = (kind == KIND_LM) ? S.lm_src[s] : s;
        const bool on = kind == KIND_LM || S.slot[s].active;
        const int d2 = d >> 1;                                   // 16-byte pieces of a row
        constexpr int kMaxPieces = 8;
        float2 xv[kMaxPieces];
        uint32_t gw[kMaxPieces];                                 // the gains do not wait for anybody
#pragma unroll
        for (int k = 0; k < kMaxPieces; ++k) {
          const int e2 = wi * 32 + lane + k * nw * 32;
          gw[k] = e2 < d2 ? __ldg(reinterpret_cast<const uint32_t*>(gain) + e2) : 0u;
        }
        {
          int n = 0;
#pragma unroll
          for (int k = 0; k < kMaxPieces; ++k) {
            if (wi * 32 + lane + k * nw * 32 < d2) n = k + 1;
            xv[k] = make_float2(0.0f, 0.0f);
          }
          const uint2* p0 = xbuf + (size_t)src * d + 2 * (wi * 32 + lane);
          if (on) {
            if (from_embed) {
              const uint32_t* er = reinterpret_cast<const uint32_t*>(A.embed + (size_t)S.slot[s].tok * d);
#pragma unroll
              for (int k = 0; k < kMaxPieces; ++k) {
                const int e2 = wi * 32 + lane + k * nw * 32;
                if (e2 < d2) { const uint32_t w2 = __ldg(er + e2); xv[k] = make_float2(__uint_as_float(w2 << 16), __uint_as_float(w2 & 0xFFFF0000u)); }
              }
            } else {
              // (four loads in flight at a time: rows of up to 4 x 64 x warps elements need one trip)
              const int n_warp = __shfl_sync(0xffffffffu, n, 0);      // lane 0 has the most pieces
#pragma unroll
              for (int k0 = 0; k0 < kMaxPieces; k0 += 4) {
                if (k0 >= n_warp) break;
                uint4 raw[4];
                const uint2* pk = p0 + (size_t)k0 * nw * 64;
                ll_poll<4>([&](int j) { return pk + (size_t)j * nw * 64; }, n - k0, ep_in, raw, S, A.err);
#pragma unroll
                for (int k = 0; k < 4; ++k) if (k0 + k < n) xv[k0 + k] = make_float2(__uint_as_float(raw[k].x), __uint_as_float(raw[k].z));
              }
            }
          }
        }
        float sq = 0.0f;
#pragma unroll
        for (int k = 0; k < kMaxPieces; ++k) sq = fmaf(xv[k].x, xv[k].x, fmaf(xv[k].y, xv[k].y, sq));
        sq = warp_sum_f32(sq);
        if (lane == 0) S.red[warp][0] = sq;
        __syncthreads();
        float tot = 0.0f;
#pragma unroll 1
        for (int w2 = s; w2 < kPW; w2 += n_in) tot += S.red[w2][0];
        const float sc = 1.0f / sqrtf(tot / (float)d + A.eps);
#pragma unroll
        for (int k = 0; k < kMaxPieces; ++k) {
          const int e2 = wi * 32 + lane + k * nw * 32;
          if (e2 < d2) {
            const uint32_t g2 = gw[k];
            *reinterpret_cast<uint32_t*>(act + s * apitch + 2 * e2) =
                pack_bf16(xv[k].x * sc * __uint_as_float(g2 << 16), xv[k].y * sc * __uint_as_float(g2 & 0xFFFF0000u));
          }
        }
        __syncthreads();
      } else if (kind == KIND_O && ka < kb) {
        // ---- stage the attention output, whole rows: put every pair's partial results together -----
        // How many partial results a (slot, KV head) pair has follows from the step's chunk geometry (the same
        // arithmetic as in the CTAs that produce them).
        // Warp w serves input row w % n_in; the row's warps walk its groups of 4 output dims.
        const int nvec = g.kchunk >> 2;
        const int s = warp % n_in, wi = warp / n_in, nw = (kPW - s + n_in - 1) / n_in;
        const int hd_shift = 31 - __clz(A.hd);                 // head size is a power of two
#pragma unroll 1
        for (int jv0 = wi * 32; jv0 < nvec; jv0 += nw * 32) {
          const int jv = jv0 + lane;
          const bool item = jv < nvec;
          const int j = item ? jv << 2 : 0;
          const int head = j >> hd_shift, dd = j - (head << hd_shift);
          const size_t base = ((size_t)s * A.H + head) * A.max_splits;
          const int n_seg = (item && S.slot[s].active) ? S.nseg[s][head] : 0;
          float4 v = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
          float M = -INFINITY, den = 0.0f;
          const int n_seg_warp = __reduce_max_sync(0xffffffffu, n_seg);
#pragma unroll 1
          for (int j0 = 0; j0 < n_seg_warp; j0 += 2) {   // running maximum over the partial results in their fixed order
            uint4 raw[6];                                 // per partial result: (max, sum), output dims dd..dd+1, dd+2..dd+3
            const int nq = max(0, min(2, n_seg - j0));
            const uint2* pml = A.part_ml + (base + j0) * 2;
            const uint2* po = A.part_o + (base + j0) * A.hd + dd;
            const int hd_ = A.hd;
            ll_poll<6>([&](int j) { const int q = j / 3, t = j - 3 * q; return t == 0 ? pml + 2 * q : po + (size_t)q * hd_ + 2 * (t - 1); },
                       3 * nq, ep_att, raw, S, A.err);
            uint4 rml[2] = {raw[0], raw[3]}, ro0[2] = {raw[1], raw[4]}, ro1[2] = {raw[2], raw[5]};
            float Mn = M;
#pragma unroll
            for (int q = 0; q < 2; ++q) if (q < nq) Mn = fmaxf(Mn, __uint_as_float(rml[q].x));
            const float fo = (M > -INFINITY) ? expf(M - Mn) : 0.0f;
            v.x *= fo; v.y *= fo; v.z *= fo; v.w *= fo; den *= fo;
#pragma unroll
            for (int q = 0; q < 2; ++q) {
              const float mq = __uint_as_float(rml[q].x);
              if (q < nq && mq > -INFINITY) {
                const float f = expf(mq - Mn);
                v.x = fmaf(f, __uint_as_float(ro0[q].x), v.x); v.y = fmaf(f, __uint_as_float(ro0[q].z), v.y);
                v.z = fmaf(f, __uint_as_float(ro1[q].x), v.z); v.w = fmaf(f, __uint_as_float(ro1[q].z), v.w);
                den = fmaf(f, __uint_as_float(rml[q].z), den);
              }
            }
            M = Mn;
          }
          if (n_seg > 0) { const float r = 1.0f / den; v.x *= r; v.y *= r; v.z *= r; v.w *= r; }
          uint2 pk;
          pk.x = pack_bf16(v.x, v.y); pk.y = pack_bf16(v.z, v.w);
          if (item) *reinterpret_cast<uint2*>(act + s * apitch + j) = pk;
        }
        __syncthreads();
      }
      TSEC(0);

      // ---- units of this CTA: rounds of kWG units, one per warp group --------------------------------
      float c[4] = {0.0f, 0.0f, 0.0f, 0.0f};
      float lm_max = -INFINITY;
      const int nsub_eff = g.nsub < kWG ? g.nsub : kWG;       // groups that share one tile in a round
#pragma unroll 1
      for (unsigned k0 = ka; k0 < kb; k0 += kWG) {
        const unsigned k = k0 + (unsigned)wgrp;
        const bool has = k < kb;
        int sub = 0;
        if (has) sub = unit_sub(S.ulist[k - ubase]);
        if (kind == KIND_DN) {
          // stage this round's chunks of the gated product (left as bf16 by the gate/up epilogue): area of
          // group w <- columns of its sub-unit, 16 bytes at a time
          // (a flagged word carries two bf16 values; a 16-byte load brings four of them).  Warp w serves the area of
          // group w / kGW; its kGW warps walk the chunk's 16-byte pieces of every input row, all loads in flight.
          const int nvec = g.kchunk >> 2;                       // 16-byte pieces of a chunk
          const int w2 = warp / kGW, part = warp - w2 * kGW;
          const unsigned kq = k0 + (unsigned)w2;
          const int sq = kq < kb ? unit_sub(S.ulist[kq - ubase]) : 0;
          int jj = part * 32 + lane, s2 = 0;                    // this lane's next (piece, row)
#pragma unroll 1
          while (__shfl_sync(0xffffffffu, jj, 0) < nvec) {      // (lane 0 has the most pieces: a warp-uniform trip count)
            const uint2* ptr[8];
            uint4 raw[8];
            int dst[8];
#pragma unroll
            for (int t = 0; t < 8; ++t) {
              ptr[t] = nullptr; dst[t] = -1;
              if (jj < nvec) {
                if (kq < kb && S.slot[s2].active) {
                  const int j = jj << 2;
                  ptr[t] = A.mid + (((size_t)s2 * A.F + (size_t)sq * g.kchunk + j) >> 1);
                  dst[t] = w2 * area_elems + s2 * apitch + j;
                }
                if (++s2 == n_in) { s2 = 0; jj += kGW * 32; }
              }
            }
            ll_poll<8>([&](int j) { return ptr[j]; }, 8, ep_gu, raw, S, A.err);
#pragma unroll
            for (int t = 0; t < 8; ++t) if (dst[t] >= 0) *reinterpret_cast<uint2*>(act + dst[t]) = make_uint2(raw[t].x, raw[t].z);
          }
          __syncthreads();
          TSEC(0);
        }
        bool landed = true;
        if (has) {
          const int slot = (int)(k % (unsigned)A.n_ring);
          landed = wait_full(S, slot, (k / (unsigned)A.n_ring) & 1u, A.err);
        }
        if (__syncthreads_or(!landed)) { alive = false; goto drain; }
        TSEC(1);
        // the residual word this thread's epilogue adds to is requested now (it arrived phases ago) and is there when
        // the products are done
        const uint2* base_p = nullptr;
        uint2 base_w = make_uint2(0u, 0u);
        if ((kind == KIND_O && layer > 0) || kind == KIND_DN) {
          const int q = tid >> 7, e = tid & 127, r = e & 15, n = e >> 4;
          const unsigned kq = k0 + (unsigned)q;
          if (kq < kb) {
            const uint32_t eq = S.ulist[kq - ubase];
            if ((q & (nsub_eff - 1)) == 0 && (unit_sub(eq) + nsub_eff == g.nsub) && n < n_in && S.slot[n].active) {
              base_p = (kind == KIND_O ? A.xa : A.x1) + (size_t)n * d + unit_tile(eq) * 16 + r;
              base_w = ll_load1(base_p);
            }
          }
        }
        if (has) {
          if (sub < kWG) { c[0] = 0.0f; c[1] = 0.0f; c[2] = 0.0f; c[3] = 0.0f; }     // first round of a tile
          const unsigned char* tile_s = ring + (size_t)(k % (unsigned)A.n_ring) * A.slot_bytes;
          const uint32_t tpitch = (uint32_t)g.kchunk * 2u + 16u;
          const __nv_bfloat16* act_g = act + ((kind == KIND_DN) ? wgrp * area_elems : 0);
          const uint32_t a_base = smem_u32(tile_s) + (uint32_t)((lane & 7) + ((lane >> 3) & 1) * 8) * tpitch + (uint32_t)(lane >> 4) * 16u;
          const uint32_t b_base = smem_u32(act_g) + (uint32_t)(lane & 7) * (uint32_t)apitch * 2u + (uint32_t)((lane >> 3) & 1) * 16u;
          const int nkb = g.kchunk >> 4;
#pragma unroll 2
          for (int kblk = wl; kblk < nkb; kblk += kGW) {
            uint32_t a[4], bfr[2];
            ldsm_x4(a, a_base + (uint32_t)kblk * 32u);
            ldsm_x2(bfr, b_base + (uint32_t)kblk * 32u);
            mma_bf16(c, a, bfr);
          }
        }
        float* cp = cpart + (size_t)((k0 / kWG) & 1u) * (kPW * 128);
        {
          const int gq = lane >> 2, tq = lane & 3;
          float* w0 = cp + warp * 128;
          *reinterpret_cast<float2*>(w0 + gq * 8 + tq * 2) = make_float2(c[0], c[1]);
          *reinterpret_cast<float2*>(w0 + (gq + 8) * 8 + tq * 2) = make_float2(c[2], c[3]);
        }
        __syncthreads();                        // slots fully read, partial tiles complete
        TSEC(2);
        cons_done = (kb < k0 + kWG) ? kb : k0 + kWG;
        // epilogue: thread (group q, row r, slot n); the first group of a tile's set sums the set's warps
        {
          const int q = tid >> 7, e = tid & 127, r = e & 15, n = e >> 4;
          const unsigned kq = k0 + (unsigned)q;
          int sq = 0, tile = 0;
          const bool on = kq < kb;
          if (on) { const uint32_t eq = S.ulist[kq - ubase]; sq = unit_sub(eq); tile = unit_tile(eq); }
          const bool lead = on && (q & (nsub_eff - 1)) == 0 && (sq + nsub_eff == g.nsub);   // tile complete in this round (nsub_eff is 1, 2 or 4)
          const bool slot_on = n < n_in && (kind == KIND_LM || S.slot[n].active);
          const int o = tile * 16 + r;
          // the residual this tile adds to: its words arrived phases ago (layer 0: the embedding itself)
          float base = 0.0f;
          if (lead && slot_on && (kind == KIND_O || kind == KIND_DN)) {
            const unsigned ep_b = kind == KIND_O ? ep_prev_dn : ep_o;
            if (kind == KIND_O && layer == 0) base = __bfloat162float(A.embed[(size_t)S.slot[n].tok * d + o]);
            else base = __uint_as_float(base_w.y == ep_b ? base_w.x : ll_wait1(base_p, ep_b, S, A.err));
          }
          float v = 0.0f;
          if (lead) {
            const int w_hi = (q + nsub_eff) * kGW;
#pragma unroll 1
            for (int w2 = q * kGW; w2 < w_hi; ++w2) v += cp[w2 * 128 + r * 8 + n];
          }
          if (kind == KIND_GU) {
            const float up = __shfl_down_sync(0xffffffffu, v, 8);
            // bf16: the down projection rounds its input to bf16 anyway; two neighbours share a flagged word
            const float gated = v / (1.0f + expf(-v)) * up;
            const float right = __shfl_down_sync(0xffffffffu, gated, 1);
            if (lead && r < 8 && (r & 1) == 0 && slot_on)
              ll_store(A.mid + (((size_t)n * A.F + tile * 8 + r) >> 1), pack_bf16(gated, right), ep_gu);
          } else if (kind == KIND_LM) {
            if (lead && slot_on && o < V) {
              A.logits_own[((size_t)step * R + n) * V + o] = v;
              lm_max = fmaxf(lm_max, v);
            }
          } else if (kind == KIND_QKV) {
            if (lead && slot_on) ll_store(A.qkv + (size_t)n * A.qkv_w + o, __float_as_uint(v), ep_qkv);
          } else {
            // residual add
            if (lead && slot_on)
              ll_store((kind == KIND_O ? A.x1 : A.xa) + (size_t)n * d + o, __float_as_uint(base + v), kind == KIND_O ? ep_o : ep_dn);
          }
        }
        // refill the slot this group has just released: after the results are on their way (the copy's issue is not
        // free), by the group's last warp, whose lanes serve the highest slot numbers and are mostly idle above
        if (has && wl == kGW - 1 && lane == 0) {
          const unsigned kn = k + (unsigned)A.n_ring;
          if (kn < total_units) issue_unit(A, S, ring, kn, per_step, pre_units);
        }
        TSEC(3);
      }
      if (kind == KIND_LM) {
        // running maxima of the logits: 16 lanes of a slot, then the CTA; every CTA publishes its maxima (0: it
        // stored no logit of the row) behind a fence, so whoever has them all may also read the logits
#pragma unroll
        for (int o2 = 8; o2 > 0; o2 >>= 1) lm_max = fmaxf(lm_max, __shfl_xor_sync(0xffffffffu, lm_max, o2));
        const int n = (tid & 127) >> 4;
        if ((tid & 15) == 0 && n < R && lm_max > -INFINITY) atomicMax(&S.lmmax[n], ord_encode(lm_max));
        __syncthreads();
        if (tid < R) {
          __threadfence();
          ll_store(A.rowmax + (size_t)cta * kPSlots + tid, S.lmmax[tid], ep_lm);
        }
      }
      // ---- attention over the rows' caches (after the QKV phase) -----------------------------------
      // The caches of all (slot, KV head) pairs are cut into chunks of split_len positions; the chunks, in
      // (slot, head, position) order, are dealt to the CTAs in contiguous ranges, so a CTA walks along one
      // cache for several chunks.  A warp keeps its positions of K and V in registers, runs its own
      // softmax and ACCUMULATES (max, sum, un-normalised output) per head in shared memory across the
      // chunks of a segment (= the part of one pair's cache this CTA owns): no block-wide exchange per
      // chunk, the next chunk's K and V are requested as soon as the registers are free.  At the end of
      // a segment the 16 warps are merged (plus the positions produced in this very phase, which come
      // from the QKV output, not from the cache) into ONE partial result (max, sum, un-normalised
      // output) per head; the partial results of a pair are put together by the O-projection phase
      // while it stages its input (every CTA needs all of it anyway), so this phase ends without a
      // second exchange between CTAs.
      // The cached positions do not depend on the QKV phase (its positions come from the QKV output),
      // so the first chunk's K and V are requested BEFORE the grid barrier and arrive while it is taken.
      const int LPR = A.hd >> 3;                     // lanes per cache row (8 bf16 per 16-byte load)
      const int PPW = 32 / LPR, PPB = kPW * PPW;     // positions per warp / per CTA pass
      const int sub = lane % LPR, pgrp = lane / LPR;
      // chunks of split_len positions (4 register passes of the CTA); short caches give fewer chunks than
      // CTAs - shorter chunks were measured slower there (the phase is latency-bound)
      const int split_len = A.split_len;
      struct Walk { int s, gk, split, nsplit, g0; };          // g0 = global index of the pair's first chunk
      auto seek = [&](int g, Walk& w) {
        int s = 0, rem = g, acc = 0, nsplit = 0;
#pragma unroll 1
        for (; s < ns; ++s) {
          nsplit = S.slot[s].active ? (S.slot[s].pos + split_len) / split_len : 0;
          if (rem < A.Hkv * nsplit) break;
          rem -= A.Hkv * nsplit; acc += A.Hkv * nsplit;
        }
        w.s = s; w.nsplit = nsplit; w.gk = nsplit ? rem / nsplit : 0; w.split = nsplit ? rem - w.gk * nsplit : 0;
        w.g0 = acc + w.gk * nsplit;
      };
      // Head size 64 with chunks of 256 positions runs on the tensor cores: a warp owns 16 positions of the chunk and
      // loads K and V straight into mma A fragments (positions, resp. dims, as rows; the heads of the group are the 8
      // columns of B).  The order of the summed index of a product is free, so the 64 dims of q.k are dealt to the
      // k-steps such that lane (g, t) needs the 16-byte pieces t and t + 4 of rows g and g + 8; in V^T P^T row g of
      // m-tile j stands for dim 8g + 2j (row g + 8 for 8g + 2j + 1), so the lane needs piece g of the four positions
      // 2t, 2t+1, 8+2t, 9+2t (pairs of positions are interleaved with byte permutes).
      const bool mma_path = (A.hd == 64) && (split_len == kPW * 16);
      const int gq = lane >> 2, t4 = lane & 3;
      auto issue_loads = [&](const Walk& w, uint4 (&kr)[4], uint4 (&vr)[4], bool want_k, bool want_v) {
        const int pos = S.slot[w.s].pos;
        const int p_lo = w.split * split_len, cnt = min(split_len, pos + 1 - p_lo);
        const int fresh_lo = pos - (w.s >= R ? 1 : 0);
        const size_t off = ((((size_t)S.slot[w.s].row * A.L + layer) * A.Hkv + w.gk) * A.cap) * A.hd;
        if (mma_path) {
          const int lim = min(cnt, fresh_lo - p_lo);                   // cached positions of the chunk: [0, lim)
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int pk = warp * 16 + (i >> 1) * 8 + gq;                // K: n-tile i/2, row g; piece t or t + 4
            const int pv = warp * 16 + (i >> 1) * 8 + 2 * t4 + (i & 1);   // V: positions 2t, 2t+1, 8+2t, 9+2t; piece g
            if (want_k) kr[i] = pk < lim ? __ldcg(reinterpret_cast<const uint4*>(A.kc + off + (size_t)(p_lo + pk) * 64 + (t4 + 4 * (i & 1)) * 8)) : make_uint4(0u, 0u, 0u, 0u);
            if (want_v) vr[i] = pv < lim ? __ldcg(reinterpret_cast<const uint4*>(A.vc + off + (size_t)(p_lo + pv) * 64 + gq * 8)) : make_uint4(0u, 0u, 0u, 0u);
          }
          return;
        }
#pragma unroll
        for (int ps = 0; ps < 4; ++ps) {
          const int p = ps * PPB + warp * PPW + pgrp;
          const bool ok = p < cnt && p_lo + p < fresh_lo;
          if (want_k) kr[ps] = ok ? __ldcg(reinterpret_cast<const uint4*>(A.kc + off + (size_t)(p_lo + p) * A.hd + sub * 8)) : make_uint4(0u, 0u, 0u, 0u);
          if (want_v) vr[ps] = ok ? __ldcg(reinterpret_cast<const uint4*>(A.vc + off + (size_t)(p_lo + p) * A.hd + sub * 8)) : make_uint4(0u, 0u, 0u, 0u);
        }
      };
      uint4 kreg[4], vreg[4];
      Walk cur{0, 0, 0, 0, 0}, nxt{0, 0, 0, 0, 0};
      int T = 0, g_lo = 0, g_hi = 0;
      PHASE_END();                                  // (its block-wide barrier also orders the geometry written at step start)
      if (kind == KIND_QKV) {
        T = S.att[0]; g_lo = S.att[1]; g_hi = S.att[2];
        cur.s = S.att[3]; cur.gk = S.att[4]; cur.split = S.att[5]; cur.nsplit = S.att[6]; cur.g0 = S.att[7];
        // the cached positions do not depend on this step's projections: their loads are in flight while the q, k, v
        // words are waited for
        if (g_lo < g_hi) issue_loads(cur, kreg, vreg, true, true);
      }

      if (kind == KIND_QKV) {
        int seg_first_split = 0;
#pragma unroll 1
        for (int g = g_lo; g < g_hi; ++g) {
          const bool have_next = g + 1 < g_hi;
          if (have_next) {
            nxt = cur; nxt.split++;
            if (nxt.split == nxt.nsplit) seek(g + 1, nxt);
          }
          const int s = cur.s, gk = cur.gk, split = cur.split, nsplit = cur.nsplit;
          const int pos = S.slot[s].pos;
          const int p_lo = split * split_len, cnt = min(split_len, pos + 1 - p_lo);
          const int fresh_lo = pos - (s >= R ? 1 : 0), n_fresh = pos - fresh_lo + 1;
          const bool seg_start = (g == g_lo) || split == 0;
          const bool seg_end = !have_next || split == nsplit - 1;
          if (seg_start) {
            seg_first_split = split;
            // stage q (all heads of the group), fresh k and v: RoPE, bf16 rounding.  One index space so
            // that every element is fetched by a different thread in one round trip.
            const int n_q = grp * half, n_k = n_fresh * half, n_v = n_fresh * A.hd;
#pragma unroll 1
            for (int idx0 = 0; idx0 < n_q + n_k + n_v; idx0 += kPT) {
              const int idx = idx0 + tid;
              const bool item = idx < n_q + n_k + n_v;
              int sj = s, col = 0, pj = pos, i = 0;
              float* dst = &S.q[0][0];
              bool pair = true;
              if (!item) {
                pair = false;
              } else if (idx < n_q) {
                const int t = idx / half; i = idx - t * half;
                sj = s; pj = pos; col = (gk * grp + t) * A.hd + i; dst = &S.q[t][i];
              } else if (idx < n_q + n_k) {
                const int j = (idx - n_q) / half; i = (idx - n_q) - j * half;
                sj = s - j * R; pj = pos - j; col = d + gk * A.hd + i; dst = &S.kf[j][i];
              } else {
                const int j = (idx - n_q - n_k) / A.hd; i = (idx - n_q - n_k) - j * A.hd;
                sj = s - j * R; pj = pos; col = d + kvd + gk * A.hd + i; dst = &S.vf[j][i]; pair = false;
              }
              const uint2* pr = A.qkv + (size_t)sj * A.qkv_w + col;
              float cs = 1.0f, sn = 0.0f, x2 = 0.0f;
              if (pair) { cs = A.rope_cos[(size_t)pj * half + i]; sn = A.rope_sin[(size_t)pj * half + i]; }
              uint32_t w1, w2;
              ll_wait1x2(item ? pr : nullptr, pair ? pr + half : nullptr, ep_qkv, w1, w2, S, A.err);          // both in flight
              const float x1 = __uint_as_float(w1);
              if (pair) x2 = __uint_as_float(w2);
              if (item) dst[0] = round_bf16(x1 * cs - x2 * sn);
              if (pair) dst[half] = round_bf16(x2 * cs + x1 * sn);
            }
            __syncthreads();
            TSEC(0);
            if (split + (g_hi - 1 - g) >= nsplit - 1 && tid < A.hd) {   // this segment reaches the pair's last split: it appends the new position
              const size_t off = ((((size_t)S.slot[s].row * A.L + layer) * A.Hkv + gk) * A.cap) * A.hd;
              A.kc[off + (size_t)pos * A.hd + tid] = __float2bfloat16_rn(S.kf[0][tid]);
              A.vc[off + (size_t)pos * A.hd + tid] = __float2bfloat16_rn(S.vf[0][tid]);
              __threadfence();        // read from the cache one step later, by CTAs that have seen this CTA's partial results
            }
          }
          if (mma_path) {
            // ---- per warp: scores, softmax, P V of its 16 positions for all heads of the group at once ----
            // The cache tile is the A operand (16 positions, resp. 16 dims, as rows), the group's heads are the 8
            // columns of B: scores^T = K q^T (4 mma), out^T = V^T P^T (8 mma with P as bf16 head + remainder).
            const int lim = min(cnt, fresh_lo - p_lo);
            uint32_t qa[4][2];
            {
              const float* qr = S.q[gq < grp ? gq : 0];
#pragma unroll
              for (int kk = 0; kk < 4; ++kk) {
                const int d0 = (kk < 2 ? 0 : 32) + 8 * t4 + 4 * (kk & 1);
                const float2 x = *reinterpret_cast<const float2*>(qr + d0), y = *reinterpret_cast<const float2*>(qr + d0 + 2);
                qa[kk][0] = gq < grp ? pack_bf16(x.x, x.y) : 0u;      // q is bf16-valued already
                qa[kk][1] = gq < grp ? pack_bf16(y.x, y.y) : 0u;
              }
            }
            // entries 0, 1: position g, heads 2t, 2t+1; entries 2, 3: position g + 8
            float sc[2][4];
            sc[0][0] = sc[0][1] = sc[0][2] = sc[0][3] = 0.0f;
            sc[1][0] = sc[1][1] = sc[1][2] = sc[1][3] = 0.0f;
            {
              const uint32_t a0[4] = {kreg[0].x, kreg[2].x, kreg[0].y, kreg[2].y}, a1[4] = {kreg[0].z, kreg[2].z, kreg[0].w, kreg[2].w};
              const uint32_t a2[4] = {kreg[1].x, kreg[3].x, kreg[1].y, kreg[3].y}, a3[4] = {kreg[1].z, kreg[3].z, kreg[1].w, kreg[3].w};
              mma_bf16(sc[0], a0, qa[0]); mma_bf16(sc[1], a1, qa[1]);
              mma_bf16(sc[0], a2, qa[2]); mma_bf16(sc[1], a3, qa[3]);
            }
            if (have_next) issue_loads(nxt, kreg, vreg, true, false);   // K registers are free
            float sv[4], mxe[2];
#pragma unroll
            for (int e = 0; e < 4; ++e)
              sv[e] = (warp * 16 + (e >> 1) * 8 + gq < lim) ? (sc[0][e] + sc[1][e]) * A.attn_scale : -INFINITY;
            mxe[0] = fmaxf(sv[0], sv[2]); mxe[1] = fmaxf(sv[1], sv[3]);
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
              mxe[0] = fmaxf(mxe[0], __shfl_xor_sync(0xffffffffu, mxe[0], o));
              mxe[1] = fmaxf(mxe[1], __shfl_xor_sync(0xffffffffu, mxe[1], o));
            }
            float pw[4], sume[2];
#pragma unroll
            for (int e = 0; e < 4; ++e) pw[e] = (sv[e] > -INFINITY) ? __expf(sv[e] - mxe[e & 1]) : 0.0f;
            sume[0] = pw[0] + pw[2]; sume[1] = pw[1] + pw[3];
            // the weights as a bf16 head and a bf16 remainder (two products, fp32 sums), moved from accumulator layout
            // (positions as rows) to B-operand layout (positions as the summed index)
            uint32_t ph[2], pl[2];
            {
              const float h0 = round_bf16(pw[0]), h1 = round_bf16(pw[1]), h2 = round_bf16(pw[2]), h3 = round_bf16(pw[3]);
              ph[0] = movmatrix_trans(pack_bf16(h0, h1)); ph[1] = movmatrix_trans(pack_bf16(h2, h3));
              pl[0] = movmatrix_trans(pack_bf16(pw[0] - h0, pw[1] - h1)); pl[1] = movmatrix_trans(pack_bf16(pw[2] - h2, pw[3] - h3));
            }
            // out^T: m-tile j, row g = dim 8g + 2j, row g + 8 = dim 8g + 2j + 1 (the lane holds piece g of its four positions)
            float oc[4][4];
            {
              const uint32_t va[4] = {vreg[0].x, vreg[0].y, vreg[0].z, vreg[0].w}, vb[4] = {vreg[1].x, vreg[1].y, vreg[1].z, vreg[1].w};
              const uint32_t vc2[4] = {vreg[2].x, vreg[2].y, vreg[2].z, vreg[2].w}, vd[4] = {vreg[3].x, vreg[3].y, vreg[3].z, vreg[3].w};
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                oc[j][0] = oc[j][1] = oc[j][2] = oc[j][3] = 0.0f;
                const uint32_t af[4] = {__byte_perm(va[j], vb[j], 0x5410u), __byte_perm(va[j], vb[j], 0x7632u),
                                        __byte_perm(vc2[j], vd[j], 0x5410u), __byte_perm(vc2[j], vd[j], 0x7632u)};
                mma_bf16(oc[j], af, ph);
                mma_bf16(oc[j], af, pl);
              }
            }
            if (have_next) issue_loads(nxt, kreg, vreg, false, true);   // ... and the V registers
#pragma unroll
            for (int o = 4; o < 32; o <<= 1) {
              sume[0] += __shfl_xor_sync(0xffffffffu, sume[0], o);
              sume[1] += __shfl_xor_sync(0xffffffffu, sume[1], o);
            }
            // accumulate into the warp's running state of this segment: the lane holds dims 8g .. 8g+7 of heads 2t, 2t+1
            float m_new[2] = {0.0f, 0.0f}, l_new[2] = {0.0f, 0.0f};
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const int head = 2 * t4 + e;
              if (head < grp) {
                float* so_w = s_o + ((size_t)warp * grp + head) * 64 + 8 * gq;
                float m_old = -INFINITY, l_old = 0.0f;
                if (!seg_start) { m_old = S.red[warp][head]; l_old = S.red2[warp][head]; }
                const float M = fmaxf(m_old, mxe[e]);
                const float f_old = (m_old > -INFINITY) ? __expf(m_old - M) : 0.0f;
                const float f_new = (mxe[e] > -INFINITY) ? __expf(mxe[e] - M) : 0.0f;
#pragma unroll
                for (int q4 = 0; q4 < 2; ++q4) {
                  float4 c4 = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                  float4* pp = reinterpret_cast<float4*>(so_w + 4 * q4);
                  if (!seg_start) { c4 = *pp; c4.x *= f_old; c4.y *= f_old; c4.z *= f_old; c4.w *= f_old; }
                  c4.x = fmaf(oc[2 * q4][e], f_new, c4.x); c4.y = fmaf(oc[2 * q4][2 + e], f_new, c4.y);
                  c4.z = fmaf(oc[2 * q4 + 1][e], f_new, c4.z); c4.w = fmaf(oc[2 * q4 + 1][2 + e], f_new, c4.w);
                  *pp = c4;
                }
                m_new[e] = M; l_new[e] = l_old * f_old + sume[e] * f_new;
              }
            }
            __syncwarp();                                  // every lane has read the old maxima and sums
            if (gq == 0) {
#pragma unroll
              for (int e = 0; e < 2; ++e)
                if (2 * t4 + e < grp) { S.red[warp][2 * t4 + e] = m_new[e]; S.red2[warp][2 * t4 + e] = l_new[e]; }
            }
            __syncwarp();
          } else
          // ---- per warp: scores, softmax, P V over its cached positions of this chunk, head by head ----
#pragma unroll 1
          for (int t = 0; t < grp; ++t) {
            float qf[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) qf[e] = S.q[t][sub * 8 + e];
            float scv[4];
            float mx = -INFINITY;
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
              const int p = ps * PPB + warp * PPW + pgrp;
              float kf8[8];
              Elem<__nv_bfloat16>::unpack(kreg[ps], kf8);
              float dd = 0.0f;
#pragma unroll
              for (int e = 0; e < 8; ++e) dd = fmaf(kf8[e], qf[e], dd);
#pragma unroll 1
              for (int o = LPR >> 1; o > 0; o >>= 1) dd += __shfl_xor_sync(0xffffffffu, dd, o);
              scv[ps] = (p < cnt && p_lo + p < fresh_lo) ? dd * A.attn_scale : -INFINITY;
              mx = fmaxf(mx, scv[ps]);
            }
            if (t == grp - 1 && have_next) issue_loads(nxt, kreg, vreg, true, false);   // K registers are free
#pragma unroll 1
            for (int o = LPR; o < 32; o <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float oacc[8], sum = 0.0f;
#pragma unroll
            for (int e = 0; e < 8; ++e) oacc[e] = 0.0f;
#pragma unroll
            for (int ps = 0; ps < 4; ++ps) {
              const float pw = (scv[ps] > -INFINITY) ? expf(scv[ps] - mx) : 0.0f;
              sum += pw;
              float vf8[8];
              Elem<__nv_bfloat16>::unpack(vreg[ps], vf8);
#pragma unroll
              for (int e = 0; e < 8; ++e) oacc[e] = fmaf(pw, vf8[e], oacc[e]);
            }
            if (t == grp - 1 && have_next) issue_loads(nxt, kreg, vreg, false, true);   // ... and the V registers
#pragma unroll 1
            for (int o = LPR; o < 32; o <<= 1) {
              sum += __shfl_xor_sync(0xffffffffu, sum, o);
#pragma unroll
              for (int e = 0; e < 8; ++e) oacc[e] += __shfl_xor_sync(0xffffffffu, oacc[e], o);
            }
            if (pgrp == 0) {
              // accumulate into the warp's running state of this segment (only this warp touches it)
              float* so_w = s_o + ((size_t)warp * grp + t) * A.hd + sub * 8;
              float m_old = -INFINITY, l_old = 0.0f;
              if (!seg_start) { m_old = S.red[warp][t]; l_old = S.red2[warp][t]; }
              const float M = fmaxf(m_old, mx);
              const float f_old = (m_old > -INFINITY) ? expf(m_old - M) : 0.0f;
              const float f_new = (mx > -INFINITY) ? expf(mx - M) : 0.0f;
#pragma unroll
              for (int e = 0; e < 8; ++e) so_w[e] = (seg_start ? 0.0f : so_w[e] * f_old) + oacc[e] * f_new;
              if (sub == 0) { S.red[warp][t] = M; S.red2[warp][t] = l_old * f_old + sum * f_new; }
            }
            __syncwarp();
          }
          TSEC(1);
          if (seg_end) {
            const int seg_lo = seg_first_split * split_len, seg_hi = p_lo + cnt;     // positions covered by the segment
            // scores of the fresh positions that fall into this segment, from the staged k
#pragma unroll 1
            for (int combo = warp; combo < grp * n_fresh; combo += kPW) {
              const int t = combo / n_fresh, j = combo - t * n_fresh;
              float dd = 0.0f;
#pragma unroll 1
              for (int i = lane; i < A.hd; i += 32) dd = fmaf(S.kf[j][i], S.q[t][i], dd);
              dd = warp_sum_f32(dd);
              const int pj = pos - j;
              if (lane == 0) S.sc[t][j] = (pj >= seg_lo && pj < seg_hi) ? dd * A.attn_scale : -INFINITY;
            }
            __syncthreads();
            // ---- merge the warps (in warp order) and the fresh positions into the segment's partial result ----
            // Its place among the pair's partial results: with at least as many chunks as CTAs every CTA owns
            // chunks, so the segments of a pair sit on consecutive CTAs; with fewer, a segment is one chunk.
            const int c_first = ((cur.g0 + 1) * NC - 1) / T;
            const int ord = (T >= NC) ? cta - c_first : split;       // (the O-projection phase works out the count itself)
#pragma unroll 1
            for (int idx = tid; idx < grp * A.hd; idx += kPT) {
              const int t = idx / A.hd, dd = idx - t * A.hd;
              float M = -INFINITY;
#pragma unroll
              for (int w2 = 0; w2 < kPW; ++w2) M = fmaxf(M, S.red[w2][t]);
              for (int j = 0; j < n_fresh; ++j) M = fmaxf(M, S.sc[t][j]);
              float v = 0.0f, l = 0.0f;
#pragma unroll
              for (int w2 = 0; w2 < kPW; ++w2) {
                const float mw = S.red[w2][t];
                const float f = (mw > -INFINITY) ? expf(mw - M) : 0.0f;
                v = fmaf(f, s_o[((size_t)w2 * grp + t) * A.hd + dd], v);
                l = fmaf(f, S.red2[w2][t], l);
              }
              for (int j = 0; j < n_fresh; ++j) {
                const float sf = S.sc[t][j];
                if (sf > -INFINITY) { const float f = expf(sf - M); v = fmaf(f, S.vf[j][dd], v); l += f; }
              }
              const int head = gk * grp + t;
              const size_t pi = ((size_t)s * A.H + head) * A.max_splits + ord;
              ll_store(A.part_o + pi * A.hd + dd, __float_as_uint(v), ep_att);
              if (dd == 0) { ll_store(A.part_ml + pi * 2, __float_as_uint(M), ep_att); ll_store(A.part_ml + pi * 2 + 1, __float_as_uint(l), ep_att); }
            }
            TSEC(2);
            __syncthreads();
            TSEC(3);
          }
          cur = nxt;
        }
        PHASE_END();
      }
    }  // phases

    if (step < 0) continue;                             // the extra pass ends with its last layer
    // ---- ensemble: exact softmax of the m rows, weighted average, draw (Algorithm 1 steps 6-7) -----
    // Three exchanges, each a table of flagged words that every CTA polls whole: every CTA's maxima of the rows
    // (published by the LM head), every CTA's integer exp sums, the mass of every chunk of q.
    {
      const float* lg = A.logits_override ? A.logits_override + (size_t)step * R * V : A.logits_own + (size_t)step * R * V;
      const bool vec = ((V & 3) == 0) && ((reinterpret_cast<uintptr_t>(lg) & 15) == 0);
      const int n_chunks = A.n_chunks;
      const unsigned ep_base = A.epoch0 + (unsigned)it * EPS;
      const unsigned ep_lm = ep_base + 5u * (unsigned)A.L + 1u, ep_max2 = ep_lm + 1u, ep_sum = ep_lm + 2u, ep_mix = ep_lm + 3u;
      const uint2* max_tab = A.rowmax;
      unsigned ep_max = ep_lm;
      if (A.logits_override) {                        // the maxima gathered by the LM head belong to other logits
        if (tid < kPSlots) S.lmmax[tid] = 0u;
        __syncthreads();
#pragma unroll 1
        for (int item = cta; item < R * n_chunks; item += NC) {
          const int row = item / n_chunks, ch = item - row * n_chunks;
          float a[kPPer];
          load4_cg(lg + (size_t)row * V, ch * kChunk + tid * kPPer, V, vec, -INFINITY, a);
          float mx = fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3]));
          mx = warp_max_f32(mx);
          if (lane == 0 && mx > -INFINITY) atomicMax(&S.lmmax[row], ord_encode(mx));
        }
        __syncthreads();
        if (tid < R) ll_store(A.rowmax2 + (size_t)cta * kPSlots + tid, S.lmmax[tid], ep_max2);
        max_tab = A.rowmax2; ep_max = ep_max2;
        PHASE_END();
      }
      // every CTA's maxima -> the rows' maxima (a maximum does not care about order)
      if (tid < kPSlots) { S.lmmax[tid] = 0u; S.row_part[tid] = 0ull; }
      __syncthreads();
#pragma unroll 1
      for (int i0 = 0; i0 < NC * R; i0 += kPT) {
        const int i = i0 + tid, c2 = i / R, row = i - c2 * R;
        uint32_t e, unused;
        ll_wait1x2(i < NC * R ? max_tab + (size_t)c2 * kPSlots + row : nullptr, nullptr, ep_max, e, unused, S, A.err);
        if (i < NC * R && e) atomicMax(&S.lmmax[row], e);
      }
      __threadfence();                                // the logits behind the flagged words
      __syncthreads();
      if (tid < R) S.rowmax_f[tid] = ord_decode(S.lmmax[tid]);
      __syncthreads();
#pragma unroll 1
      for (int item = cta; item < R * n_chunks; item += NC) {
        const int row = item / n_chunks, ch = item - row * n_chunks;
        const int v0 = ch * kChunk + tid * kPPer;
        float a[kPPer];
        load4_cg(lg + (size_t)row * V, v0, V, vec, -INFINITY, a);
        const float mx = S.rowmax_f[row];
        unsigned long long sm = 0;
#pragma unroll
        for (int j = 0; j < kPPer; ++j) if (v0 + j < V) sm += mass_of(xexp(__fsub_rn(a[j], mx)));
        sm = block_sum_u64_p(sm, S);
        if (tid == 0) S.row_part[row] += sm;
      }
      __syncthreads();
      if (tid < R) {
        const unsigned long long t = S.row_part[tid];
        uint2* dst = A.rowsum + ((size_t)cta * kPSlots + tid) * 2;
        ll_store(dst, (uint32_t)t, ep_sum); ll_store(dst + 1, (uint32_t)(t >> 32), ep_sum);
      }
      PHASE_END();
      // every CTA's sums -> the rows' normalisers (integer sums: order-free)
      if (tid < kPSlots) S.row_part[tid] = 0ull;
      __syncthreads();
#pragma unroll 1
      for (int i0 = 0; i0 < NC * R; i0 += kPT) {
        const int i = i0 + tid, c2 = i / R, row = i - c2 * R;
        const uint4 w4 = ll_wait2(i < NC * R ? A.rowsum + ((size_t)c2 * kPSlots + row) * 2 : nullptr, ep_sum, S, A.err);
        const unsigned long long t = (unsigned long long)w4.x | ((unsigned long long)w4.z << 32);
        if (i < NC * R && t) atomicAdd(&S.row_part[row], t);
      }
      __syncthreads();
#pragma unroll 1
      for (int item = cta; item < B * n_chunks; item += NC) {
        const int b = item / n_chunks, ch = item - b * n_chunks;
        const int v0 = ch * kChunk + tid * kPPer;
        float acc[kPPer];
        float* qk_b = A.qk + ((size_t)b * G + step) * m * V;
        __syncthreads();
        if (tid < m) {
          const int row = b * m + tid;
          S.mix_mx[tid] = S.rowmax_f[row];
          S.mix_sn[tid] = norm_of(S.row_part[row]);
          S.mix_w[tid] = A.w[row];
        }
        float nxt[kPPer];
        load4_cg(lg + (size_t)(b * m) * V, v0, V, vec, -INFINITY, nxt);
        __syncthreads();
#pragma unroll 1
        for (int k = 0; k < m; ++k) {
          float a[kPPer];
#pragma unroll
          for (int j = 0; j < kPPer; ++j) a[j] = nxt[j];
          if (k + 1 < m) load4_cg(lg + (size_t)(b * m + k + 1) * V, v0, V, vec, -INFINITY, nxt);
          const float mxk = S.mix_mx[k], snk = S.mix_sn[k], wkk = S.mix_w[k];
#pragma unroll
          for (int j = 0; j < kPPer; ++j) {
            a[j] = __fdiv_rn(xexp(__fsub_rn(a[j], mxk)), snk);
            const float t = __fmul_rn(wkk, a[j]);
            acc[j] = (k == 0) ? t : __fadd_rn(acc[j], t);
          }
          store4(qk_b + (size_t)k * V, v0, V, (V & 3) == 0, a);
        }
        store4(A.q + ((size_t)b * G + step) * V, v0, V, (V & 3) == 0, acc);
        uint2* cm_dst = A.chunk_mass + ((size_t)b * n_chunks + ch) * 2;
        if (!A.greedy) {
          unsigned long long sm = 0;
#pragma unroll
          for (int j = 0; j < kPPer; ++j) if (v0 + j < V) sm += mass_of(acc[j]);
          sm = block_sum_u64_p(sm, S);                  // (its barriers: every thread's part of q is stored)
          if (tid == 0) {
            __threadfence();                            // q before the word that announces it
            ll_store(cm_dst, (uint32_t)sm, ep_mix); ll_store(cm_dst + 1, (uint32_t)(sm >> 32), ep_mix);
          }
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
#pragma unroll 1
            for (int i = 1; i < kPW; ++i)
              if (S.bestv[i] > bv || (S.bestv[i] == bv && S.besti[i] < bi)) { bv = S.bestv[i]; bi = S.besti[i]; }
            __threadfence();
            ll_store(cm_dst, __float_as_uint(bv), ep_mix); ll_store(cm_dst + 1, (uint32_t)bi, ep_mix);
          }
        }
      }
      PHASE_END();
      // every CTA locates the drawn token itself (the next step's embedding gather needs it)
#pragma unroll 1
      for (int b = 0; b < B; ++b) {
        if (A.greedy) {
          float bv = -1.0f; int bi = 0x7fffffff;
#pragma unroll 1
          for (int c0 = 0; c0 < n_chunks; c0 += kPT) {
            const int c2 = c0 + tid;
            const uint4 w4 = ll_wait2(c2 < n_chunks ? A.chunk_mass + ((size_t)b * n_chunks + c2) * 2 : nullptr, ep_mix, S, A.err);
            const float cv = __uint_as_float(w4.x);
            const int ci = (int)w4.z;
            if (c2 < n_chunks && (cv > bv || (cv == bv && ci < bi))) { bv = cv; bi = ci; }
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
#pragma unroll 1
            for (int i = 1; i < kPW; ++i)
              if (S.bestv[i] > bv || (S.bestv[i] == bv && S.besti[i] < bi)) { bv = S.bestv[i]; bi = S.besti[i]; }
            S.tok[b] = bi;
          }
          __syncthreads();
          continue;
        }
        const uint2* cm = A.chunk_mass + (size_t)b * n_chunks * 2;
        // chunk masses in parallel into shared memory, then one thread walks them
        unsigned long long T = 0;
#pragma unroll 1
        for (int c0 = 0; c0 < n_chunks; c0 += kPT) {
          unsigned long long mine = 0ull;
          {
            const uint4 w4 = ll_wait2(c0 + tid < n_chunks ? cm + (size_t)(c0 + tid) * 2 : nullptr, ep_mix, S, A.err);
            if (c0 + tid < n_chunks) mine = (unsigned long long)w4.x | ((unsigned long long)w4.z << 32);
          }
          if (n_chunks <= kPT && tid < n_chunks) S.cm[tid] = mine;       // one trip to L2 serves the sum and the walk
          T += block_sum_u64_p(mine, S);
        }
        __threadfence();                              // q behind the words that announce it
        __syncthreads();
        if (tid == 0) {
          S.result = 0x7fffffff;
          if (T == 0ull) { atomicOr(A.err, 1); S.chunk = -1; }
          else {
            const unsigned long long thr = draw_threshold(A.u[b * G + step], T);
            int c2 = 0;
            unsigned long long pre = 0;
#pragma unroll 1
            for (; c2 < n_chunks - 1; ++c2) {
              unsigned long long mc;
              if (n_chunks <= kPT) mc = S.cm[c2];
              else { const uint4 w4 = ll_load2(cm + (size_t)c2 * 2); mc = (unsigned long long)w4.x | ((unsigned long long)w4.z << 32); }   // (seen valid above)
              const unsigned long long nx = pre + mc;
              if (nx > thr) break;
              pre = nx;
            }
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
#pragma unroll 1
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
#undef PHASE_END
#undef TSEC
  return;

drain:
  // a wait ran out: let the copies already issued land before the shared memory is released.
  // Units below cons_done have been consumed; every consumed unit k had unit k + n_ring issued.
  if (tid == 0) {
    unsigned hi = cons_done + (unsigned)A.n_ring;
    if (hi > total_units) hi = total_units;
#pragma unroll 1
    for (unsigned k = cons_done; k < hi; ++k) {
      const int slot = (int)(k % (unsigned)A.n_ring);
      const unsigned parity = (k / (unsigned)A.n_ring) & 1u;
      unsigned spins = 0;
      while (!mbar_try_wait(&S.full[slot], parity) && ++spins < kSpinLimit) __nanosleep(64);
    }
  }
  __syncthreads();
}

}  // namespace tabed
