// C boundary of the TABED round: handle, state, launch sequences.  See include/tabed.h for the
// contract of every entry point; the kernels live in forward_kernels.cuh / decide_kernels.cuh.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <new>
#include <type_traits>
#include <utility>
#include <vector>

#include "../../include/tabed.h"
#include "exact_math.cuh"
#include "forward_kernels.cuh"
#include "decide_kernels.cuh"
#include "round_kernel.cuh"
#include "gemm_tc.cuh"
#include "attn_tc.cuh"
#include "request_kernels.cuh"

using namespace tabed;

namespace {

enum Phase { PH_IDLE = 0, PH_DRAFTED = 1, PH_VERIFIED = 2 };

constexpr int kMaxDevices = 64;       // device ordinals the per-device tables below can hold

struct DeviceGuard {
  int prev = -1; bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

struct tabed_handle {
  tabed_config cfg;
  bool has_drafter = false;
  cudaStream_t stream = nullptr;
  int R = 0, B = 0, m = 0, G = 0, V = 0, d = 0, F = 0, H = 0, Hkv = 0, hd = 0, L = 0, cap = 0;
  int D = 1, Rt = 0;                // token tree: candidates per depth; target rows per request G + 1 + G (D - 1)
  int *cand = nullptr, *acc_prim = nullptr, *sib_tok = nullptr;   // [B][G][D] candidates; [B] accepted primaries; [B] sibling token
  int n_dev = 0, n_chunks = 0, ns = 1, max_splits = 0, qkv_w = 0;
  size_t esz = 4;
  // drafter (caller-owned device memory)
  const void *embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  std::vector<const void*> wq, wk, wv, wo, w_gate, w_up, w_down, norm1, norm2;
  // library-owned device memory
  std::vector<void*> allocs;
  void *kc = nullptr, *vc = nullptr;
  float *rope_cos = nullptr, *rope_sin = nullptr;
  int *kv_len = nullptr, *pending = nullptr;
  float *w = nullptr;
  long long *dev = nullptr, *ring = nullptr, *running = nullptr, *pushed = nullptr;
  int *req_ticket = nullptr, *row_flag = nullptr;     // scratch of the per-request cluster kernels
  int *ring_head = nullptr, *ring_count = nullptr, *grid_j = nullptr;
  SlotDesc* slots = nullptr; int* last_slot = nullptr;
  float *x = nullptr, *qkv = nullptr, *attn_out = nullptr, *mid = nullptr, *part_o = nullptr, *part_ml = nullptr;
  float *logits_own = nullptr, *qk = nullptr, *q = nullptr, *p = nullptr, *scratch_q = nullptr;
  int *tokens = nullptr, *n_accept = nullptr, *next_token = nullptr, *w_argmax = nullptr;
  unsigned long long* chunk_mass = nullptr; ChunkBest* chunk_best = nullptr;
  int* err = nullptr;
  int cs_max = 8;                   // largest cluster the per-request kernels may use on this device (8 portable, 16 opt-in)
  int cs_active[5] = {0, 0, 0, 0, 0};   // clusters of 1, 2, 4, 8, 16 CTAs that the device keeps resident at once
  bool req_dyn_ok = false;          // the cluster kernels may take up to kReqDynSmemMax of dynamic shared memory
  int cta_budget = 3;               // CTAs per SM a launch of the per-request kernels may have in total (3, 6, 12 measured: 3 best)
  // staging for the host-buffer entry point
  float *st_u_draft = nullptr, *st_u_accept = nullptr, *st_u_resid = nullptr, *st_target = nullptr;
  int* st_tokens = nullptr;
  // host-side state
  int phase = PH_IDLE;
  bool round_has_forward = false;
  bool cand_is_tokens = false;      // the round's candidates are its tokens (drafted by the persistent kernel: chains only)
  const float* logits_override = nullptr;   // tabed_debug_override_logits
  const float* u_policy = nullptr;          // tabed_set_policy_uniforms (random weight policy)
  std::vector<int> len_ub;          // upper bound of every row's committed length
  std::vector<int> pend_cnt;        // pending tokens of every request as the host last saw them
  bool pend_known = false;          // ... and whether that is still what the device holds
  int64_t launches = 0;
  // persistent drafting-round kernel (bf16 drafters with at most kPSlots slots per step)
  bool persist_ok = false;
  int path_sel = 0;                 // 0 auto, 1 per-operation kernels, 2 persistent kernel
  RoundArgs ra{};                   // everything that does not change between rounds
  int n_cta = 0; size_t persist_smem = 0;
  unsigned launches_persist = 0;
  LayerW* layer_tab = nullptr;
  // its exchange buffers of flagged words {value, epoch} and the epoch the next launch starts from
  uint2 *ll_xa = nullptr, *ll_x1 = nullptr, *ll_qkv = nullptr, *ll_mid = nullptr, *ll_po = nullptr, *ll_pml = nullptr;
  uint2 *ll_rowmax = nullptr, *ll_rowmax2 = nullptr, *ll_rowsum = nullptr, *ll_cmass = nullptr;
  std::vector<std::pair<void*, size_t>> ll_all;       // every exchange buffer (cleared when the epoch counter wraps)
  unsigned ll_epoch = 0;
  uint2* ll_probe = nullptr;        // a word nobody ever writes (tabed_debug_barrier_timeout)
  // tensor-core streaming attention of the per-operation paths (bf16 caches, head size 64)
  int* attn_tickets = nullptr; int n_sm = 0;
  bool atc_ok = false; CUtensorMap tm_k, tm_v;
  unsigned char* packed = nullptr;
  unsigned long long* trace = nullptr; int trace_stride = 0; bool trace_on = false; int trace_cta = 0;
  // tensor-core projections for many rows (bf16 drafter, more than 8 slots per step)
  bool tc_ok = false;                        // tcgen05 projections are set up (prefill in chunks; drafting when tc_auto)
  bool tc_auto = false;                      // ... and are the automatic choice for drafting (no persistent kernel)
  int slot_cap = 0;                          // slots the step buffers hold: 2R, or a prefill chunk if that is more
  struct TcKind { int rows, K, m_tiles, k_chunks, ks, cps; size_t bytes; };
  TcKind tck[5]{};                  // KIND_QKV, KIND_O, KIND_GU (gate|up rows), KIND_DN, KIND_LM
  unsigned char* tc_w = nullptr;    // [L][QKV | O | GU | DN] then LM, operand blocks of k_pack_tc
  size_t tc_layer_stride = 0, tc_off[5]{};
  unsigned char* tc_act = nullptr;  // activation operand blocks of the group being projected
  float *tc_pq = nullptr, *tc_po = nullptr, *tc_pgu = nullptr, *tc_pd = nullptr;   // k-split partials [ks][2R][rows]
  size_t tc_smem = 0;
  // per-kernel-class timing (tabed_profile_begin / tabed_profile_end)
  int prof_class = -1;
  std::vector<cudaEvent_t> prof_events;     // start/stop pairs
  // tabed_round_host: the target's logits (by far the largest input) travel on a stream of the library's own while
  // the drafting runs on the caller's; the two events order that copy after the caller's earlier work and before
  // the verification
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_round_begin = nullptr, ev_target_ready = nullptr;
  size_t prof_used = 0;
};

namespace {

// Records a start/stop event pair on the handle's stream around the launches of one kernel class.
struct ProfScope {
  tabed_handle* h; bool on;
  ProfScope(tabed_handle* hh, int cls) : h(hh), on(hh->prof_class == cls) { if (on) rec(); }
  ~ProfScope() { if (on) rec(); }
  void rec() {
    if (h->prof_used == h->prof_events.size()) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
      h->prof_events.push_back(e);
    }
    cudaEventRecord(h->prof_events[h->prof_used++], h->stream);
  }
};

#define TABED_LAUNCH(h, kern, grid, block, smem, ...)                 \
  do {                                                                \
    kern<<<(grid), (block), (smem), (h)->stream>>>(__VA_ARGS__);      \
    (h)->launches++;                                                  \
  } while (0)

// Launch as a programmatic dependent of the kernel before it in the stream (the kernel calls pdl_wait before it
// touches anything dynamic): launch latency and prologue overlap the predecessor's tail.
template <typename... KArgs, typename... Args>
void launch_pdl(tabed_handle* h, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = h->stream;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, KArgs(std::forward<Args>(args))...);
  h->launches++;
}
#define TABED_LAUNCH_PDL(h, kern, grid, block, smem, ...) launch_pdl((h), (kern), dim3(grid), dim3(block), (smem), __VA_ARGS__)

// `n_clusters` clusters of `cs` CTAs, as a programmatic dependent of the kernel before it in the stream.
constexpr size_t kReqDynSmemMax = 64u * 1024u;      // slices kept in shared memory by the softmax passes (two CTAs per SM still fit)

template <typename ArgT>
void launch_request_clusters(tabed_handle* h, void (*kern)(ArgT), int n_clusters, int cs, const ArgT& args, size_t dyn_smem = 0) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(n_clusters * cs)); cfg.blockDim = dim3(kReqThreads); cfg.dynamicSmemBytes = dyn_smem; cfg.stream = h->stream;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = (unsigned)cs; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 2;
  cudaLaunchKernelEx(&cfg, kern, args);
  h->launches++;
}

// CTAs per cluster: as many as the budget of CTAs per SM over all clusters allows, no finer than ~1024
// vocabulary elements per CTA; slice = vocabulary elements per CTA (a multiple of 4, so that slices start on
// 16-byte boundaries).
int pick_cluster(const tabed_handle* h, int n_clusters, int* slice, int budget_scale = 1) {
  const int by_v = (h->V + 1023) / 1024, n_sm = h->n_sm > 0 ? h->n_sm : 148;
  int cs = 1;
  // (measured on 32 requests: many small CTAs in several waves beat one wave of large ones - the passes are bound by
  // dependent latencies and arithmetic, and more resident warps hide both)
  while (cs * 2 <= h->cs_max && (long long)n_clusters * cs * 2 <= (long long)h->cta_budget * budget_scale * n_sm && cs < by_v) cs *= 2;
  *slice = ((h->V + cs - 1) / cs + 3) & ~3;
  return cs;
}

template <typename T>
int dev_alloc(tabed_handle* h, T** out, size_t count, bool zero = true) {
  void* ptr = nullptr;
  const size_t bytes = std::max<size_t>(count, 1) * sizeof(T);
  if (cudaMalloc(&ptr, bytes) != cudaSuccess) { cudaGetLastError(); return TABED_ERR_CUDA; }
  h->allocs.push_back(ptr);
  if (zero && cudaMemsetAsync(ptr, 0, bytes, h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  *out = reinterpret_cast<T*>(ptr);
  return TABED_OK;
}

int pick_ns(int n) {            // accumulator columns per weight pass
  const int opts[] = {1, 2, 3, 4, 6, 8};
  for (int o : opts) if (o >= std::min(n, 8)) return o;
  return 8;
}

// ---- projection dispatch ---------------------------------------------------------------------
template <typename T, int NS, int RPW, int EPI>
void launch_gemv_inst(tabed_handle* h, const GemvArgs& a, int n_chunks) {
  constexpr bool ROUND_IN = !std::is_same<T, float>::value;
  auto kern = k_gemv<T, NS, RPW, EPI, ROUND_IN>;
  const size_t smem = (size_t)NS * a.K * sizeof(float);
  static bool attr_set[kMaxDevices] = {false};          // the attribute belongs to a (function, device) pair
  if (!attr_set[h->cfg.device]) {
    cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
    attr_set[h->cfg.device] = true;
  }
  const int n_out = (EPI == EPI_SWIGLU) ? a.rows0 : (a.rows0 + a.rows1 + a.rows2);
  const int n_groups = (n_out + RPW - 1) / RPW;
  const int ctas = std::max(1, std::min((n_groups + kGemvWarps - 1) / kGemvWarps, 148 * 8));
  TABED_LAUNCH(h, kern, dim3(ctas, n_chunks), kGemvThreads, smem, a);
}

template <typename T, int NS, int EPI>
void launch_gemv_rpw(tabed_handle* h, const GemvArgs& a, int n_chunks) {
  const int n_out = (EPI == EPI_SWIGLU) ? a.rows0 : (a.rows0 + a.rows1 + a.rows2);
  const int per_row = (EPI == EPI_SWIGLU) ? 2 : 1;
  const int warps_full = 148 * kGemvWarps * 2;
  if constexpr (NS <= 4 && EPI != EPI_SWIGLU) {
    if (n_out >= warps_full * 4) { launch_gemv_inst<T, NS, 4, EPI>(h, a, n_chunks); return; }
  }
  if constexpr (NS <= 4 || EPI != EPI_SWIGLU) {
    if (n_out >= warps_full * 2) { launch_gemv_inst<T, NS, 2, EPI>(h, a, n_chunks); return; }
  }
  (void)per_row;
  launch_gemv_inst<T, NS, 1, EPI>(h, a, n_chunks);
}

template <typename T, int EPI>
void launch_gemv_ns(tabed_handle* h, const GemvArgs& a, int ns) {
  const int n_chunks = (a.n_slots + ns - 1) / ns;
  switch (ns) {
    case 1: launch_gemv_rpw<T, 1, EPI>(h, a, n_chunks); break;
    case 2: launch_gemv_rpw<T, 2, EPI>(h, a, n_chunks); break;
    case 3: launch_gemv_rpw<T, 3, EPI>(h, a, n_chunks); break;
    case 4: launch_gemv_rpw<T, 4, EPI>(h, a, n_chunks); break;
    case 6: launch_gemv_rpw<T, 6, EPI>(h, a, n_chunks); break;
    default: launch_gemv_rpw<T, 8, EPI>(h, a, n_chunks); break;
  }
}

void launch_gemv(tabed_handle* h, const GemvArgs& a, int epi, int ns) {
  const bool f32 = h->cfg.dtype == TABED_DTYPE_FP32;
  if (epi == EPI_STORE) { if (f32) launch_gemv_ns<float, EPI_STORE>(h, a, ns); else launch_gemv_ns<__nv_bfloat16, EPI_STORE>(h, a, ns); }
  else if (epi == EPI_RESID) { if (f32) launch_gemv_ns<float, EPI_RESID>(h, a, ns); else launch_gemv_ns<__nv_bfloat16, EPI_RESID>(h, a, ns); }
  else { if (f32) launch_gemv_ns<float, EPI_SWIGLU>(h, a, ns); else launch_gemv_ns<__nv_bfloat16, EPI_SWIGLU>(h, a, ns); }
}

// act_out != null (and *wrote_act given): the caller wants the output as the next projection's bf16 operand blocks;
// the kernel that can do that sets *wrote_act, otherwise the fp32 rows in h->attn_out are the result.
template <typename T, int HD>
void launch_attention_hd(tabed_handle* h, int layer, int n_slots, int max_pos, unsigned char* act_out, int act_npad, bool* wrote_act) {
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    // bandwidth-oriented kernel: all K, V loads of a split in flight at once
    const int split_len = attn_bw_split_len(HD);
    const int splits = std::max(1, (max_pos + split_len - 1) / split_len);
    const int grp = h->H / h->Hkv;
    const size_t smem = ((size_t)(kAttnBwThreads / 32) * grp * (HD + 2)) * sizeof(float);
    auto part = k_attn_split_bf16<HD>;
    static bool attr_set[kMaxDevices] = {false};
    if (!attr_set[h->cfg.device]) { cudaFuncSetAttribute(part, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024); attr_set[h->cfg.device] = true; }
    if constexpr (HD == kAtcHd) {
      if (h->atc_ok && n_slots <= kAtcMaxSlots) {
        // fixed grid of streaming CTAs, contiguous chunk ranges, TMA-fed tensor-core arithmetic, in-kernel merge
        // two CTAs per SM with three stages each when the shared memory allows, else one CTA with a deeper ring
        // per stage: the K and V tiles, q of the cache, and one set of the eight warps' states
        const size_t seg_state = (size_t)kAtcWarps * grp * (HD + 2) * sizeof(float);      // the eight warps' states of a segment
        const size_t per_stage = 2 * (size_t)kAtcTile + (size_t)grp * HD * sizeof(float) + seg_state;
        int n_ctas = std::min(kAtcMaxCtas, 2 * h->n_sm), n_stages = 3;
        if (1024 + n_stages * per_stage + seg_state > 108u * 1024u) {
          n_ctas = std::min(kAtcMaxCtas, h->n_sm);
          n_stages = (int)std::min<size_t>(kAtcMaxStages, (kAtcMaxDynSmem - 1024u - seg_state) / per_stage);
        }
        if (n_stages >= 3) {
          const size_t smem2 = 1024 + n_stages * per_stage + seg_state;       // one more set of states than stages
          static bool attr2_set[kMaxDevices] = {false};
          if (!attr2_set[h->cfg.device]) { cudaFuncSetAttribute(k_attn_tc_bf16, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAtcMaxDynSmem); attr2_set[h->cfg.device] = true; }
          AttnTcArgs a;
          a.qkv = h->qkv; a.slots = h->slots; a.n_slots = n_slots; a.H = h->H; a.Hkv = h->Hkv; a.layer = layer; a.L = h->L;
          a.cap = h->cap; a.qkv_w = h->qkv_w; a.part_o = h->part_o; a.part_ml = h->part_ml; a.max_splits = h->max_splits;
          a.act_out = act_out; a.act_npad = act_npad;
          a.tickets = h->attn_tickets; a.out = h->attn_out; a.scale = 1.0f / sqrtf((float)h->hd); a.err = h->err; a.n_stages = n_stages;
          TABED_LAUNCH_PDL(h, k_attn_tc_bf16, n_ctas, kAtcThreads, smem2, h->tm_k, h->tm_v, a);
          if (wrote_act) *wrote_act = act_out != nullptr;
          return;
        }
      }
    }
    if (smem <= 96 * 1024) {
      TABED_LAUNCH(h, part, dim3(splits, h->Hkv, n_slots), kAttnBwThreads, smem, h->qkv, h->slots, h->H, h->Hkv,
                   reinterpret_cast<const __nv_bfloat16*>(h->kc), reinterpret_cast<const __nv_bfloat16*>(h->vc), layer, h->L, h->cap,
                   h->part_o, h->part_ml, h->max_splits, 1.0f / sqrtf((float)h->hd));
      auto merge = k_attn_merge<HD>;
      TABED_LAUNCH(h, merge, dim3(h->H, n_slots), HD, 0, h->slots, h->H, split_len, h->part_o, h->part_ml, h->max_splits, h->attn_out);
      return;
    }
  }
  const int split_len = (max_pos > 2048) ? 256 : 128;
  const int splits = std::max(1, (max_pos + split_len - 1) / split_len);
  const float scale = 1.0f / sqrtf((float)h->hd);
  auto part = k_attn_partial<T, HD>;
  auto merge = k_attn_merge<HD>;
  TABED_LAUNCH(h, part, dim3(splits, h->Hkv, n_slots), kAttnThreads, 0, h->qkv, h->slots, h->H, h->Hkv,
               reinterpret_cast<const T*>(h->kc), reinterpret_cast<const T*>(h->vc), layer, h->L, h->cap, split_len,
               h->part_o, h->part_ml, h->max_splits, scale);
  TABED_LAUNCH(h, merge, dim3(h->H, n_slots), HD, 0, h->slots, h->H, split_len, h->part_o, h->part_ml,
               h->max_splits, h->attn_out);
}

template <typename T>
void launch_attention_t(tabed_handle* h, int layer, int n_slots, int max_pos, unsigned char* act_out = nullptr, int act_npad = 0,
                        bool* wrote_act = nullptr) {
  if (wrote_act) *wrote_act = false;
  switch (h->hd) {
    case 32: launch_attention_hd<T, 32>(h, layer, n_slots, max_pos, act_out, act_npad, wrote_act); break;
    case 64: launch_attention_hd<T, 64>(h, layer, n_slots, max_pos, act_out, act_npad, wrote_act); break;
    default: launch_attention_hd<T, 128>(h, layer, n_slots, max_pos, act_out, act_npad, wrote_act); break;
  }
}

// One shared-weight decoder step over `n_slots` slots.  max_pos: host upper bound of (position+1).
void run_step(tabed_handle* h, StepArgs sa, int n_slots, int max_pos, float* logits_out) {
  const bool f32 = h->cfg.dtype == TABED_DTYPE_FP32;
  sa.R = h->R; sa.m = h->m; sa.d = h->d; sa.G = h->G;
  sa.kv_len = h->kv_len; sa.pending = h->pending;
  sa.slots = h->slots; sa.last_slot = h->last_slot; sa.x = h->x; sa.err = h->err; sa.kv_capacity = h->cap;
  if (f32) TABED_LAUNCH(h, k_begin_step<float>, n_slots, 128, 0, sa, reinterpret_cast<const float*>(h->embed));
  else TABED_LAUNCH(h, k_begin_step<__nv_bfloat16>, n_slots, 128, 0, sa, reinterpret_cast<const __nv_bfloat16*>(h->embed));
  const int ns = (sa.mode == STEP_PREFILL) ? 1 : h->ns;
  const int kvd = h->Hkv * h->hd;
  for (int l = 0; l < h->L; ++l) {
    GemvArgs a{};
    a.W0 = h->wq[l]; a.W1 = h->wk[l]; a.W2 = h->wv[l]; a.rows0 = h->d; a.rows1 = kvd; a.rows2 = kvd;
    a.K = h->d; a.in = h->x; a.in_stride = h->d; a.gain = h->norm1[l]; a.eps = h->cfg.rms_eps;
    a.out = h->qkv; a.out_stride = h->qkv_w; a.slots = h->slots; a.n_slots = n_slots;
    { ProfScope ps(h, TABED_PROF_QKV); launch_gemv(h, a, EPI_STORE, ns); }
    ProfScope* pa = new ProfScope(h, TABED_PROF_ATTENTION);
    if (f32) {
      TABED_LAUNCH(h, k_rope_append<float>, n_slots, 128, 0, h->qkv, h->slots, h->H, h->Hkv, h->hd, h->rope_cos,
                   h->rope_sin, reinterpret_cast<float*>(h->kc), reinterpret_cast<float*>(h->vc), l, h->L, h->cap);
      launch_attention_t<float>(h, l, n_slots, max_pos);
    } else {
      TABED_LAUNCH(h, k_rope_append<__nv_bfloat16>, n_slots, 128, 0, h->qkv, h->slots, h->H, h->Hkv, h->hd,
                   h->rope_cos, h->rope_sin, reinterpret_cast<__nv_bfloat16*>(h->kc),
                   reinterpret_cast<__nv_bfloat16*>(h->vc), l, h->L, h->cap);
      launch_attention_t<__nv_bfloat16>(h, l, n_slots, max_pos);
    }
    delete pa;
    GemvArgs o{};
    o.W0 = h->wo[l]; o.rows0 = h->d; o.K = h->H * h->hd; o.in = h->attn_out; o.in_stride = h->H * h->hd;
    o.out = h->x; o.out_stride = h->d; o.slots = h->slots; o.n_slots = n_slots;
    { ProfScope ps(h, TABED_PROF_OPROJ); launch_gemv(h, o, EPI_RESID, ns); }
    GemvArgs gu{};
    gu.W0 = h->w_gate[l]; gu.W1 = h->w_up[l]; gu.rows0 = h->F; gu.rows1 = h->F; gu.K = h->d;
    gu.in = h->x; gu.in_stride = h->d; gu.gain = h->norm2[l]; gu.eps = h->cfg.rms_eps;
    gu.out = h->mid; gu.out_stride = h->F; gu.slots = h->slots; gu.n_slots = n_slots;
    { ProfScope ps(h, TABED_PROF_GATEUP); launch_gemv(h, gu, EPI_SWIGLU, ns); }
    GemvArgs dn{};
    dn.W0 = h->w_down[l]; dn.rows0 = h->d; dn.K = h->F; dn.in = h->mid; dn.in_stride = h->F;
    dn.out = h->x; dn.out_stride = h->d; dn.slots = h->slots; dn.n_slots = n_slots;
    { ProfScope ps(h, TABED_PROF_DOWN); launch_gemv(h, dn, EPI_RESID, ns); }
  }
  if (logits_out) {
    GemvArgs hd{};
    hd.W0 = h->lm_head; hd.rows0 = h->V; hd.K = h->d; hd.in = h->x; hd.in_stride = h->d;
    hd.src_slot = h->last_slot; hd.gain = h->final_norm; hd.eps = h->cfg.rms_eps;
    hd.out = logits_out; hd.out_stride = h->V; hd.slots = nullptr; hd.n_slots = h->R;
    ProfScope ps(h, TABED_PROF_LM_HEAD);
    launch_gemv(h, hd, EPI_STORE, h->ns);
  }
}

// Algorithm 1 steps 6-7 for all requests on logits [B][m][V]: one launch, one cluster per request.
void run_ensemble(tabed_handle* h, const float* logits, const float* w, const float* u, int u_stride,
                  int* y0, int y0_stride, int* y1, int y1_stride, float* qk_out, long long qk_stride,
                  float* q_out, long long q_stride, int n_cand = 1, int* cand = nullptr, int cand_stride = 0) {
  ProfScope ps(h, TABED_PROF_ENSEMBLE);
  EnsembleArgs a{};
  const int cs = pick_cluster(h, h->B, &a.slice);
  a.V = h->V; a.m = h->m; a.greedy = h->cfg.sample_mode == TABED_MODE_GREEDY;
  a.logits = logits; a.w = w; a.u = u; a.u_stride = u_stride;
  a.qk_out = qk_out; a.qk_req_stride = qk_stride; a.q_out = q_out; a.q_req_stride = q_stride;
  a.out0 = y0; a.out0_stride = y0_stride; a.out1 = y1; a.out1_stride = y1_stride; a.err = h->err;
  a.D = n_cand; a.cand = cand; a.cand_stride = cand_stride;
  // the CTA's slices of the m rows stay in shared memory between the softmax passes when they fit
  size_t dyn = (size_t)h->m * a.slice * sizeof(float);
  if (dyn <= kReqDynSmemMax && h->req_dyn_ok) a.ebuf_pitch = a.slice; else dyn = 0;
  launch_request_clusters(h, k_ensemble_req, h->B, cs, a, dyn);
}

// ---- persistent drafting-round kernel: geometry and set-up -----------------------------------------
// Cut a [16*n_tiles][K] weight matrix into tiles of 16 rows; a tile whose rows are longer than kcap
// becomes nsub sub-units (1, 2 or a multiple of 4, so that they line up with the 4 warp groups).
PhaseGeom pick_geom(int n_tiles, int K, int kcap) {
  const int nkb = K / 16;
  for (int nsub = 1; nsub <= 64; nsub = (nsub < 4) ? nsub * 2 : nsub + 4) {
    if (nkb % nsub || K / nsub > kcap) continue;
    return PhaseGeom{n_tiles, nsub, K / nsub, n_tiles * nsub};
  }
  return PhaseGeom{n_tiles, 0, 0, 0};
}

// Decides whether the handle's drafter can run on the persistent kernel and allocates its buffers.
int setup_persistent(tabed_handle* h) {
  const tabed_config& c = h->cfg;
  h->persist_ok = false;
  if (c.dtype != TABED_DTYPE_BF16 || h->D > 1) return TABED_OK;      // (the in-kernel draw proposes one candidate per step)
  const int grp = h->H / h->Hkv;
  // up to kPSlots / 2 rows both pending tokens of a fully accepted block share the first step's weight pass (2 R slots);
  // with more rows (up to kPSlots) the first of them gets a pass of its own, which needs two layers for its cache
  // writes to be ordered before the first step's reads
  const bool prepass = 2 * h->R > kPSlots;
  if (h->R > kPSlots || (prepass && h->L < 2) || h->B > kPSlots || h->d % 16 || h->d > kPMaxD || h->F % 16 || (h->Hkv * h->hd) % 16 ||
      grp > kMaxGroup || grp * h->hd > 512 || h->L > kPMaxL || h->H > kPMaxHeads || (h->cap + 127) / 128 > kAttnSplitMax)
    return TABED_OK;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess) return TABED_ERR_CUDA;
  if (!prop.cooperativeLaunch) return TABED_OK;
  cudaFuncAttributes fa;
  if (cudaFuncGetAttributes(&fa, k_draft_round<true>) != cudaSuccess) return TABED_ERR_CUDA;
  const int n_cta = prop.multiProcessorCount;
  if (n_cta > kPT) return TABED_OK;
  RoundArgs& A = h->ra;
  // QKV, O, gate/up and LM head rows are d_model long and stay whole; only the down projection is cut
  A.geom[KIND_QKV] = pick_geom(h->qkv_w / 16, h->d, h->d);
  A.geom[KIND_O] = pick_geom(h->d / 16, h->H * h->hd, h->d);
  A.geom[KIND_GU] = pick_geom(h->F / 8, h->d, h->d);
  A.geom[KIND_DN] = pick_geom(h->d / 16, h->F, std::max(h->d, 512));
  A.geom[KIND_LM] = pick_geom((h->V + 15) / 16, h->d, h->d);
  int kmax = 0;
  long per_step = 0;                                  // upper bound of one CTA's units per decoder step
  for (int k = 0; k < 5; ++k) {
    if (A.geom[k].nsub == 0) return TABED_OK;
    kmax = std::max(kmax, A.geom[k].kchunk);
    per_step += (long)((A.geom[k].n_tiles + n_cta - 1) / n_cta) * A.geom[k].nsub * (k == KIND_LM ? 1 : h->L);
  }
  if (per_step > kMaxUnits) return TABED_OK;
  {
    // the staging of a whole input row: its warps keep at most 8 pieces of 16 bytes per lane in flight
    const int act_slots = prepass ? h->R : 2 * h->R, warps_per_row = kPW / act_slots;
    if ((h->d / 2 + warps_per_row * 32 - 1) / (warps_per_row * 32) > 8) return TABED_OK;
  }
  A.slot_bytes = 16 * (kmax * 2 + 16);
  A.act_slots = prepass ? h->R : 2 * h->R;
  A.prepass = prepass ? 1 : 0;
  const int dn_areas = std::min(A.geom[KIND_DN].nsub, kWG);
  const size_t act_raw = std::max((size_t)A.act_slots * (h->d + 8) * 2, (size_t)dn_areas * A.act_slots * (A.geom[KIND_DN].kchunk + 8) * 2);
  A.act_bytes = (int)((act_raw + 127) / 128 * 128);
  const size_t u_bytes = std::max<size_t>((size_t)A.act_bytes + 2 * kPW * 128 * sizeof(float), (size_t)kPW * 512 * sizeof(float));
  const size_t avail = (size_t)prop.sharedMemPerBlockOptin - fa.sharedSizeBytes - 1024;
  if (avail < u_bytes + (size_t)kWG * A.slot_bytes) return TABED_OK;      // a round needs kWG units in flight
  A.n_ring = (int)std::min<size_t>(kPRing, (avail - u_bytes) / A.slot_bytes);
  h->persist_smem = (size_t)A.n_ring * A.slot_bytes + u_bytes;
  // (the device's opt-in maximum, not this handle's own size: a later handle with a smaller ring must not lower it)
  const int persist_attr = (int)((size_t)prop.sharedMemPerBlockOptin - fa.sharedSizeBytes);
  if (cudaFuncSetAttribute(k_draft_round<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, persist_attr) != cudaSuccess ||
      cudaFuncSetAttribute(k_draft_round<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, persist_attr) != cudaSuccess)
    return TABED_ERR_CUDA;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_draft_round<true>, kPT, h->persist_smem) != cudaSuccess) return TABED_ERR_CUDA;
  if (per_sm < 1) return TABED_OK;
  h->n_cta = n_cta;

  int rc = TABED_OK;
  auto A2 = [&](auto** ptr, size_t count) { if (rc == TABED_OK) rc = dev_alloc(h, ptr, count); };
  const size_t d = h->d;
  A2(&h->layer_tab, (size_t)h->L);
  auto LL = [&](uint2** ptr, size_t count) {
    if (rc == TABED_OK) rc = dev_alloc(h, ptr, count);           // zeroed: no launch ever stamps epoch 0
    if (rc == TABED_OK) h->ll_all.push_back({*ptr, std::max<size_t>(count, 1) * sizeof(uint2)});
  };
  LL(&h->ll_xa, kPSlots * d); LL(&h->ll_x1, kPSlots * d); LL(&h->ll_qkv, (size_t)kPSlots * h->qkv_w);
  LL(&h->ll_mid, (size_t)kPSlots * h->F / 2);
  LL(&h->ll_po, (size_t)kPSlots * h->H * h->max_splits * h->hd); LL(&h->ll_pml, (size_t)kPSlots * h->H * h->max_splits * 2);
  LL(&h->ll_rowmax, (size_t)n_cta * kPSlots); LL(&h->ll_rowmax2, (size_t)n_cta * kPSlots); LL(&h->ll_rowsum, (size_t)n_cta * kPSlots * 2);
  LL(&h->ll_cmass, (size_t)h->B * h->n_chunks * 2); LL(&h->ll_probe, 2);
  // private copy of the weights, unit by unit (one contiguous block per bulk copy)
  size_t unit_bytes[5], kind_bytes[5];
  for (int k = 0; k < 5; ++k) {
    unit_bytes[k] = 16 * ((size_t)A.geom[k].kchunk * 2 + 16);
    kind_bytes[k] = unit_bytes[k] * A.geom[k].n_units;
  }
  A.pack_off[KIND_QKV] = 0;
  A.pack_off[KIND_O] = A.pack_off[KIND_QKV] + kind_bytes[KIND_QKV];
  A.pack_off[KIND_GU] = A.pack_off[KIND_O] + kind_bytes[KIND_O];
  A.pack_off[KIND_DN] = A.pack_off[KIND_GU] + kind_bytes[KIND_GU];
  A.pack_layer_stride = A.pack_off[KIND_DN] + kind_bytes[KIND_DN];
  A.pack_off[KIND_LM] = A.pack_layer_stride * h->L;
  if (rc == TABED_OK) {
    void* ptr = nullptr;
    if (cudaMalloc(&ptr, A.pack_off[KIND_LM] + kind_bytes[KIND_LM]) != cudaSuccess) { cudaGetLastError(); return TABED_OK; }   // no room: per-operation path
    h->allocs.push_back(ptr);
    h->packed = reinterpret_cast<unsigned char*>(ptr);
  }
  h->trace_stride = 5 * h->L + 8;
  A2(&h->trace, (size_t)h->G * h->trace_stride * kTraceRec);
  if (rc != TABED_OK) return rc;
  std::vector<LayerW> tab(h->L);
  using bf = __nv_bfloat16;
  for (int l = 0; l < h->L; ++l)
    tab[l] = LayerW{(const bf*)h->wq[l], (const bf*)h->wk[l], (const bf*)h->wv[l], (const bf*)h->wo[l], (const bf*)h->w_gate[l],
                    (const bf*)h->w_up[l], (const bf*)h->w_down[l], (const bf*)h->norm1[l], (const bf*)h->norm2[l]};
  if (cudaMemcpyAsync(h->layer_tab, tab.data(), tab.size() * sizeof(LayerW), cudaMemcpyHostToDevice, h->stream) != cudaSuccess)
    return TABED_ERR_CUDA;
  const int kvd = h->Hkv * h->hd;
  for (int l = 0; l <= h->L; ++l) {
    for (int k = 0; k < 5; ++k) {
      if ((l == h->L) != (k == KIND_LM)) continue;
      PackArgs P{};
      P.kind = k; P.g = A.geom[k];
      P.dst = h->packed + A.pack_off[k] + (k == KIND_LM ? 0 : (size_t)l * A.pack_layer_stride);
      if (k == KIND_QKV) { P.w0 = tab[l].wq; P.w1 = tab[l].wk; P.w2 = tab[l].wv; P.rows0 = h->d; P.rows1 = kvd; P.rows2 = kvd; P.K = h->d; }
      else if (k == KIND_O) { P.w0 = tab[l].wo; P.rows0 = h->d; P.K = h->H * h->hd; }
      else if (k == KIND_GU) { P.w0 = tab[l].wg; P.w1 = tab[l].wu; P.rows0 = h->F; P.rows1 = h->F; P.K = h->d; }
      else if (k == KIND_DN) { P.w0 = tab[l].wd; P.rows0 = h->d; P.K = h->F; }
      else { P.w0 = (const bf*)h->lm_head; P.rows0 = h->V; P.K = h->d; }
      k_pack_units<<<A.geom[k].n_units, 256, 0, h->stream>>>(P);
    }
  }
  if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  A.layers = h->layer_tab; A.embed = (const bf*)h->embed; A.final_norm = (const bf*)h->final_norm;
  A.rope_cos = h->rope_cos; A.rope_sin = h->rope_sin;
  A.L = h->L; A.d = h->d; A.F = h->F; A.H = h->H; A.Hkv = h->Hkv; A.hd = h->hd; A.V = h->V; A.cap = h->cap; A.qkv_w = h->qkv_w;
  A.eps = c.rms_eps; A.attn_scale = 1.0f / sqrtf((float)h->hd);
  A.R = h->R; A.B = h->B; A.m = h->m; A.G = h->G; A.greedy = c.sample_mode == TABED_MODE_GREEDY;
  A.kv_len = h->kv_len; A.pending = h->pending; A.kc = (bf*)h->kc; A.vc = (bf*)h->vc;
  A.xa = h->ll_xa; A.x1 = h->ll_x1; A.qkv = h->ll_qkv; A.mid = h->ll_mid;
  A.part_o = h->ll_po; A.part_ml = h->ll_pml; A.max_splits = h->max_splits;
  A.logits_own = h->logits_own; A.w = h->w; A.qk = h->qk; A.q = h->q;
  A.rowmax = h->ll_rowmax; A.rowmax2 = h->ll_rowmax2; A.rowsum = h->ll_rowsum; A.chunk_mass = h->ll_cmass;
  A.n_chunks = h->n_chunks; A.tokens = h->tokens; A.err = h->err; A.packed = h->packed;
  A.trace_stride = h->trace_stride;
  h->persist_ok = true;
  return TABED_OK;
}

int launch_persistent_round(tabed_handle* h, const float* u_draft, int32_t* out_tokens, int max_pos) {
  RoundArgs A = h->ra;
  A.u = u_draft; A.out_tokens = out_tokens; A.logits_override = h->logits_override;
  (void)max_pos;
  A.split_len = (h->hd <= 64) ? 256 : 128;          // positions per attention item: 4 register passes of the CTA
  // epochs: this launch stamps epoch0 + 1 ... epoch0 + (G [+ 1]) (5 L + 8); when the counter nears its end the buffers are cleared
  const unsigned span = (unsigned)(h->G + (A.prepass ? 1 : 0)) * (5u * (unsigned)h->L + 8u);
  if (h->ll_epoch > 0xFFFFFFFFu - 2u * span) {
    for (auto& b : h->ll_all) if (cudaMemsetAsync(b.first, 0, b.second, h->stream) != cudaSuccess) return TABED_ERR_CUDA;
    h->ll_epoch = 0;
  }
  A.epoch0 = h->ll_epoch;
  h->ll_epoch += span;
  A.trace = h->trace_on ? h->trace : nullptr; A.trace_cta = h->trace_cta;
  void* args[] = {&A};
  const void* kern = h->trace_on ? (const void*)k_draft_round<true> : (const void*)k_draft_round<false>;
  if (cudaLaunchCooperativeKernel(kern, dim3(h->n_cta), dim3(kPT), args, h->persist_smem, h->stream) != cudaSuccess)
    return TABED_ERR_CUDA;
  h->launches_persist++;
  h->launches++;
  return TABED_OK;
}

// ---- tensor-core path for many rows -----------------------------------------------------------------
int setup_tc(tabed_handle* h) {
  const tabed_config& c = h->cfg;
  h->tc_ok = false;
  if (c.dtype != TABED_DTYPE_BF16 || h->slot_cap < kPrefillChunk || h->d % 8 || h->F % 8 || (h->H * h->hd) % 8) return TABED_OK;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, c.device) != cudaSuccess) return TABED_ERR_CUDA;
  if (prop.major < 10) return TABED_OK;
  const int n_sm = prop.multiProcessorCount, kvd = h->Hkv * h->hd;
  const int rows[5] = {h->qkv_w, h->d, 2 * h->F, h->d, h->V};
  const int Ks[5] = {h->d, h->H * h->hd, h->d, h->F, h->d};
  for (int k = 0; k < 5; ++k) {
    tabed_handle::TcKind& t = h->tck[k];
    t.rows = rows[k]; t.K = Ks[k];
    t.m_tiles = (t.rows + kTcM - 1) / kTcM; t.k_chunks = (t.K + kTcKC - 1) / kTcKC;
    int ks = std::max(1, std::min(std::min(t.k_chunks, 8), (n_sm + t.m_tiles - 1) / t.m_tiles));   // at most 8 slabs to sum
    if (k == KIND_LM) ks = 1;                       // logits are stored directly
    t.cps = (t.k_chunks + ks - 1) / ks;
    t.ks = (t.k_chunks + t.cps - 1) / t.cps;
    t.bytes = (size_t)t.m_tiles * t.k_chunks * tc_block_bytes(kTcM);
  }
  h->tc_off[KIND_QKV] = 0;
  h->tc_off[KIND_O] = h->tck[KIND_QKV].bytes;
  h->tc_off[KIND_GU] = h->tc_off[KIND_O] + h->tck[KIND_O].bytes;
  h->tc_off[KIND_DN] = h->tc_off[KIND_GU] + h->tck[KIND_GU].bytes;
  h->tc_layer_stride = h->tc_off[KIND_DN] + h->tck[KIND_DN].bytes;
  h->tc_off[KIND_LM] = h->tc_layer_stride * h->L;
  const int n_pad_max = (std::min(h->slot_cap, kTcMaxN) + 15) / 16 * 16;
  h->tc_smem = 0;
  for (int np = 16; np <= n_pad_max; np += 16)
    h->tc_smem = std::max(h->tc_smem, (size_t)tc_stages(np) * (tc_block_bytes(kTcM) + tc_block_bytes(np)) + 1024);
  if (h->tc_smem > (size_t)prop.sharedMemPerBlockOptin) return TABED_OK;
  if (cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)h->tc_smem) != cudaSuccess) return TABED_ERR_CUDA;
  int rc = TABED_OK;
  auto A2 = [&](auto** ptr, size_t count) { if (rc == TABED_OK) rc = dev_alloc(h, ptr, count, false); };
  const size_t S2 = (size_t)h->slot_cap;
  int kc_max = 0;
  for (int k = 0; k < 5; ++k) kc_max = std::max(kc_max, h->tck[k].k_chunks);
  A2(&h->tc_w, h->tc_off[KIND_LM] + h->tck[KIND_LM].bytes);
  A2(&h->tc_act, (size_t)kc_max * tc_block_bytes(n_pad_max));
  A2(&h->tc_pq, (size_t)h->tck[KIND_QKV].ks * S2 * h->qkv_w); A2(&h->tc_po, (size_t)h->tck[KIND_O].ks * S2 * h->d);
  A2(&h->tc_pgu, (size_t)h->tck[KIND_GU].ks * S2 * 2 * h->F); A2(&h->tc_pd, (size_t)h->tck[KIND_DN].ks * S2 * h->d);
  if (rc != TABED_OK) return rc;
  using bf = __nv_bfloat16;
  for (int l = 0; l <= h->L; ++l) {
    for (int k = 0; k < 5; ++k) {
      if ((l == h->L) != (k == KIND_LM)) continue;
      const tabed_handle::TcKind& t = h->tck[k];
      unsigned char* dst = h->tc_w + h->tc_off[k] + (k == KIND_LM ? 0 : (size_t)l * h->tc_layer_stride);
      const dim3 grid(t.k_chunks, t.m_tiles);
      if (k == KIND_QKV) k_pack_tc<<<grid, 256, 0, h->stream>>>((const bf*)h->wq[l], h->d, (const bf*)h->wk[l], kvd, (const bf*)h->wv[l], kvd, t.K, t.k_chunks, dst);
      else if (k == KIND_O) k_pack_tc<<<grid, 256, 0, h->stream>>>((const bf*)h->wo[l], h->d, nullptr, 0, nullptr, 0, t.K, t.k_chunks, dst);
      else if (k == KIND_GU) k_pack_tc<<<grid, 256, 0, h->stream>>>((const bf*)h->w_gate[l], h->F, (const bf*)h->w_up[l], h->F, nullptr, 0, t.K, t.k_chunks, dst);
      else if (k == KIND_DN) k_pack_tc<<<grid, 256, 0, h->stream>>>((const bf*)h->w_down[l], h->d, nullptr, 0, nullptr, 0, t.K, t.k_chunks, dst);
      else k_pack_tc<<<grid, 256, 0, h->stream>>>((const bf*)h->lm_head, h->V, nullptr, 0, nullptr, 0, t.K, t.k_chunks, dst);
    }
  }
  if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  h->tc_ok = true;
  h->tc_auto = !h->persist_ok;            // measured faster than one kernel per operation from 6 rows on (1.46 vs 2.20 ms)
  return TABED_OK;
}

// one tensor-core projection of a slot group whose operand blocks are already in h->tc_act
void launch_gemm_tc(tabed_handle* h, int kind, int layer, int n, float* partial, size_t slab, const SlotDesc* slots, int rows_valid) {
  const tabed_handle::TcKind& t = h->tck[kind];
  TcGemmArgs G{};
  G.a_packed = h->tc_w + h->tc_off[kind] + (kind == KIND_LM ? 0 : (size_t)layer * h->tc_layer_stride);
  G.b_packed = h->tc_act; G.partial = partial; G.slab = slab; G.slots = slots;
  G.rows_total = t.rows; G.rows_valid = rows_valid; G.n_pad = (n + 15) / 16 * 16; G.n_slots = n;
  G.k_chunks = t.k_chunks; G.ks = t.ks; G.cps = t.cps; G.err = h->err;
  G.kc = kTcKC; G.n_stages = tc_stages(G.n_pad);
  // More tiles than SMs (the LM head): stages of half a block, so that two CTAs share an SM and one's epilogue
  // overlaps the other's copies (32000 x 768 for 96 slots: 28.8 -> 23.3 us); the projections with at most one CTA
  // per SM are no faster with half stages (measured with 3, 4 and 6 of them).
  if (t.m_tiles * t.ks > h->n_sm && G.n_pad <= 128) { G.kc = kTcKC / 2; G.n_stages = 3; }
  const size_t smem = (size_t)G.n_stages * (tc_block_bytes(kTcM) + tc_block_bytes(G.n_pad)) / (kTcKC / G.kc) + 1024;
  TABED_LAUNCH_PDL(h, k_gemm_tc, t.m_tiles * t.ks, kTcThreads, smem, G);
}

// One shared-weight decoder step over `n_slots` slots with the projections on the tensor cores.
void run_step_tc(tabed_handle* h, StepArgs sa, int n_slots, int max_pos, float* logits_out) {
  using bf = __nv_bfloat16;
  sa.R = h->R; sa.m = h->m; sa.d = h->d; sa.G = h->G;
  sa.kv_len = h->kv_len; sa.pending = h->pending;
  sa.slots = h->slots; sa.last_slot = h->last_slot; sa.x = h->x; sa.err = h->err; sa.kv_capacity = h->cap;
  TABED_LAUNCH_PDL(h, k_begin_step<bf>, n_slots, 128, 0, sa, reinterpret_cast<const bf*>(h->embed));
  const size_t S2 = (size_t)h->slot_cap;
  const int d = h->d, HD = h->H * h->hd, F = h->F;
  struct Grp { int s0, n; };
  std::vector<Grp> groups;                       // up to 256 slots share one pass over the weights
  for (int g0 = 0; g0 < n_slots; g0 += kTcMaxN) groups.push_back({g0, std::min(kTcMaxN, n_slots - g0)});
  auto prep_row = [&](const Grp& g, const float* partial, int ks, size_t slab, int write_back, const void* gain, const int* src, const SlotDesc* slots) {
    PrepRowArgs P{};
    P.x = h->x; P.d = d; P.partial = partial; P.ks = partial ? ks : 0; P.slab = slab; P.src_slot = src; P.slots = slots;
    P.gain = reinterpret_cast<const bf*>(gain); P.eps = h->cfg.rms_eps; P.slot0 = g.s0; P.n = g.n; P.n_pad = (g.n + 15) / 16 * 16;
    P.write_back = write_back; P.dst = h->tc_act;
    TABED_LAUNCH_PDL(h, k_prep_row, g.n, 256, 0, P);
  };
  for (int l = 0; l < h->L; ++l) {
    {
      ProfScope ps(h, TABED_PROF_QKV);
      for (const Grp& g : groups) {
        prep_row(g, l == 0 ? nullptr : h->tc_pd, h->tck[KIND_DN].ks, S2 * d, 1, h->norm1[l], nullptr, h->slots);
        launch_gemm_tc(h, KIND_QKV, l, g.n, h->tc_pq + (size_t)g.s0 * h->qkv_w, S2 * h->qkv_w, h->slots + g.s0, h->qkv_w);
      }
      // the split-K slabs of the projection are summed by the kernel that rotates q, k and appends k, v
      TABED_LAUNCH_PDL(h, k_rope_append<bf>, n_slots, 512, 0, h->qkv, h->slots, h->H, h->Hkv, h->hd, h->rope_cos, h->rope_sin,
                   reinterpret_cast<bf*>(h->kc), reinterpret_cast<bf*>(h->vc), l, h->L, h->cap,
                   (const float*)h->tc_pq, h->tck[KIND_QKV].ks, S2 * h->qkv_w);
    }
    bool attn_wrote_act = false;
    {
      ProfScope ps(h, TABED_PROF_ATTENTION);       // the attention kernel(s) alone on this path
      // one slot group: the attention kernel can leave its output as the O projection's operand blocks
      const bool one = groups.size() == 1;
      launch_attention_t<bf>(h, l, n_slots, max_pos, one ? h->tc_act : nullptr, one ? (groups[0].n + 15) / 16 * 16 : 0, &attn_wrote_act);
    }
    {
      ProfScope ps(h, TABED_PROF_OPROJ);
      for (const Grp& g : groups) {
        const int n_pad = (g.n + 15) / 16 * 16;
        if (!attn_wrote_act)
          TABED_LAUNCH_PDL(h, k_prep_act, h->tck[KIND_O].k_chunks, 256, 0, h->attn_out + (size_t)g.s0 * HD, HD, g.n, n_pad, HD,
                     (const float*)nullptr, (const bf*)nullptr, h->tc_act);
        launch_gemm_tc(h, KIND_O, l, g.n, h->tc_po + (size_t)g.s0 * d, S2 * d, h->slots + g.s0, d);
      }
    }
    {
      ProfScope ps(h, TABED_PROF_GATEUP);
      for (const Grp& g : groups) {
        prep_row(g, h->tc_po, h->tck[KIND_O].ks, S2 * d, 1, h->norm2[l], nullptr, h->slots);
        launch_gemm_tc(h, KIND_GU, l, g.n, h->tc_pgu + (size_t)g.s0 * 2 * F, S2 * 2 * F, h->slots + g.s0, 2 * F);
      }
    }
    {
      ProfScope ps(h, TABED_PROF_DOWN);
      for (const Grp& g : groups) {
        const int n_pad = (g.n + 15) / 16 * 16;
        TABED_LAUNCH_PDL(h, k_swiglu_prep, dim3(h->tck[KIND_DN].k_chunks, g.n), kTcKC / 8, 0, h->tc_pgu, h->tck[KIND_GU].ks, S2 * 2 * F, F,
                     h->slots, g.s0, n_pad, h->tc_act);
        launch_gemm_tc(h, KIND_DN, l, g.n, h->tc_pd + (size_t)g.s0 * d, S2 * d, h->slots + g.s0, d);
      }
    }
  }
  if (logits_out) {
    ProfScope ps(h, TABED_PROF_LM_HEAD);
    for (int r0 = 0; r0 < h->R; r0 += kTcMaxN) {
      const Grp g{r0, std::min(kTcMaxN, h->R - r0)};
      prep_row(g, h->tc_pd, h->tck[KIND_DN].ks, S2 * d, 0, h->final_norm, h->last_slot, nullptr);
      launch_gemm_tc(h, KIND_LM, 0, g.n, logits_out + (size_t)r0 * h->V, 0, nullptr, h->V);
    }
  }
}

int check_cuda() { return cudaGetLastError() == cudaSuccess ? TABED_OK : TABED_ERR_CUDA; }

// Bits of the device-side error word -> return code (most severe first): a bounded wait that ran out, a cache
// position beyond the capacity, a distribution without mass (non-finite logits) or a draw that found no token.
int map_device_error(int bits) {
  if (bits & (PERR_BARRIER | PERR_COPY)) return TABED_ERR_TIMEOUT;
  if (bits & PERR_KV) return TABED_ERR_KV_OVERFLOW;
  if (bits & 3) return TABED_ERR_NUMERIC;
  return bits ? TABED_ERR_CUDA : TABED_OK;
}

// Copies the error word back, clears it on the device and synchronises the stream.
int read_clear_device_error(int* err_dev, cudaStream_t st, int* bits_out) {
  int bits = 0;
  if (cudaMemcpyAsync(&bits, err_dev, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(err_dev, 0, sizeof(int), st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess) {
    cudaGetLastError();
    return TABED_ERR_CUDA;
  }
  *bits_out = bits;
  return TABED_OK;
}

// drafting steps outside the persistent kernel: tensor-core projections when chosen (or automatic with many rows)
bool use_tc(const tabed_handle* h) {
  return h->tc_ok && (h->path_sel == TABED_PATH_TENSOR_CORE || (h->path_sel == TABED_PATH_AUTO && h->tc_auto));
}

int max_len_ub(const tabed_handle* h) {
  int mx = 0;
  for (int v : h->len_ub) mx = std::max(mx, v);
  return mx;
}

}  // namespace

// =================================================================================================
extern "C" {

const char* tabed_strerror(int code) {
  switch (code) {
    case TABED_OK: return "ok";
    case TABED_ERR_INVALID_ARG: return "invalid argument";
    case TABED_ERR_NULL_PTR: return "null pointer";
    case TABED_ERR_BAD_STATE: return "call out of order for the handle's state";
    case TABED_ERR_KV_OVERFLOW: return "row cache capacity would be exceeded";
    case TABED_ERR_CUDA: return "CUDA runtime error";
    case TABED_ERR_TIMEOUT: return "device-side wait ran out";
    case TABED_ERR_UNSUPPORTED: return "unsupported configuration";
    case TABED_ERR_NUMERIC: return "a distribution had no mass (non-finite logits)";
    default: return "unknown error code";
  }
}

int tabed_init(const tabed_config* cfg, const tabed_weights* wts, tabed_handle** out) {
  if (!cfg || !out) return TABED_ERR_NULL_PTR;
  *out = nullptr;
  const tabed_config& c = *cfg;
  if (c.vocab < 2 || c.n_inputs < 1 || c.n_inputs > TABED_MAX_INPUTS || c.n_requests < 1 || c.gamma < 1 ||
      c.gamma > 16 || c.window_h < 0 || c.window_h > 64 || c.policy < 0 || c.policy > TABED_POLICY_ADABOOST || c.distance < 0 ||
      c.distance > 1 || c.sample_mode < 0 || c.sample_mode > 1 || !(c.tau > 0.0f) || c.device < 0 || c.tree_width < 0 ||
      c.tree_width > TABED_MAX_TREE_WIDTH)
    return TABED_ERR_INVALID_ARG;
  if ((c.policy == TABED_POLICY_GRID_MT || c.policy == TABED_POLICY_GRID_HARD) && c.n_inputs != 2) return TABED_ERR_INVALID_ARG;
  if ((long long)c.n_requests * c.n_inputs > 4096) return TABED_ERR_UNSUPPORTED;
  if (wts) {
    if (c.n_layers < 1 || c.d_model < 8 || c.n_heads < 1 || c.n_kv_heads < 1 || c.d_ffn < 8 || c.kv_capacity < 1 ||
        c.dtype < 0 || c.dtype > 1 || !(c.rms_eps > 0.0f) || !(c.rope_theta > 0.0f))
      return TABED_ERR_INVALID_ARG;
    if (c.d_model % c.n_heads || c.n_heads % c.n_kv_heads || c.d_model % 8 || c.d_ffn % 8) return TABED_ERR_INVALID_ARG;
    const int hd = c.d_model / c.n_heads;
    if (hd != 32 && hd != 64 && hd != 128) return TABED_ERR_INVALID_ARG;
    if (!wts->embed || !wts->lm_head || !wts->final_norm || !wts->wq || !wts->wk || !wts->wv || !wts->wo ||
        !wts->w_gate || !wts->w_up || !wts->w_down || !wts->norm1 || !wts->norm2)
      return TABED_ERR_NULL_PTR;
    for (int l = 0; l < c.n_layers; ++l)
      if (!wts->wq[l] || !wts->wk[l] || !wts->wv[l] || !wts->wo[l] || !wts->w_gate[l] || !wts->w_up[l] ||
          !wts->w_down[l] || !wts->norm1[l] || !wts->norm2[l])
        return TABED_ERR_NULL_PTR;
    // the projection kernels read the drafter with 128-bit loads
    auto misaligned = [](const void* ptr) { return (reinterpret_cast<uintptr_t>(ptr) & 15u) != 0; };
    if (misaligned(wts->embed) || misaligned(wts->lm_head) || misaligned(wts->final_norm)) return TABED_ERR_INVALID_ARG;
    for (int l = 0; l < c.n_layers; ++l)
      if (misaligned(wts->wq[l]) || misaligned(wts->wk[l]) || misaligned(wts->wv[l]) || misaligned(wts->wo[l]) ||
          misaligned(wts->w_gate[l]) || misaligned(wts->w_up[l]) || misaligned(wts->w_down[l]) || misaligned(wts->norm1[l]) ||
          misaligned(wts->norm2[l]))
        return TABED_ERR_INVALID_ARG;
  }
  if (c.device >= kMaxDevices) return TABED_ERR_INVALID_ARG;
  int n_devices = 0;
  if (cudaGetDeviceCount(&n_devices) != cudaSuccess || c.device >= n_devices) { cudaGetLastError(); return TABED_ERR_CUDA; }
  DeviceGuard guard(c.device);
  if (!guard.ok) return TABED_ERR_CUDA;

  tabed_handle* h = new (std::nothrow) tabed_handle();
  if (!h) return TABED_ERR_CUDA;
  h->cfg = c; h->stream = reinterpret_cast<cudaStream_t>(c.stream);
  h->B = c.n_requests; h->m = c.n_inputs; h->R = h->B * h->m; h->G = c.gamma; h->V = c.vocab;
  h->D = std::max(1, c.tree_width); h->Rt = h->G + 1 + h->G * (h->D - 1);
  h->n_dev = (c.policy == TABED_POLICY_GRID_MT || c.policy == TABED_POLICY_GRID_HARD) ? kGridCand : h->m;
  h->n_chunks = (h->V + kChunk - 1) / kChunk;
  h->ns = pick_ns(h->R);
  h->has_drafter = wts != nullptr;
  int rc = TABED_OK;
  {
    cudaDeviceProp pr;
    if (cudaGetDeviceProperties(&pr, c.device) == cudaSuccess) h->n_sm = pr.multiProcessorCount;
    // the per-request cluster kernels: clusters of 16 CTAs where the device can place one (non-portable size)
    h->cs_max = 8;
    h->req_dyn_ok = cudaFuncSetAttribute(k_ensemble_req, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kReqDynSmemMax) == cudaSuccess &&
                    cudaFuncSetAttribute(k_verify_req, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kReqDynSmemMax) == cudaSuccess;
    if (cudaFuncSetAttribute(k_ensemble_req, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(k_verify_req, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(k_verify_tail, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
        cudaFuncSetAttribute(k_update_req, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(kReqMaxCluster); lc.blockDim = dim3(kReqThreads);
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = kReqMaxCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.attrs = at; lc.numAttrs = 1;
      int n16 = 0;
      bool ok = true;
      for (const void* fn : {(const void*)k_ensemble_req, (const void*)k_verify_req, (const void*)k_verify_tail, (const void*)k_update_req})
        ok = ok && cudaOccupancyMaxActiveClusters(&n16, fn, &lc) == cudaSuccess && n16 >= 1;
      if (ok) h->cs_max = kReqMaxCluster;
      // how many clusters of each size fit at once (the most demanding of the three kernels): a launch is sized for one wave
      for (int i = 0; i < 5; ++i) {
        const int cs = 1 << i;
        if (cs > h->cs_max) break;
        lc.gridDim = dim3(cs); at[0].val.clusterDim.x = cs;
        int best = 1 << 30;
        for (const void* fn : {(const void*)k_ensemble_req, (const void*)k_verify_req, (const void*)k_verify_tail, (const void*)k_update_req}) {
          int n = 0;
          if (cudaOccupancyMaxActiveClusters(&n, fn, &lc) != cudaSuccess) n = 0;
          best = std::min(best, n);
        }
        h->cs_active[i] = best;
      }
    }
    cudaGetLastError();
  }
  auto A = [&](auto** ptr, size_t count) { if (rc == TABED_OK) rc = dev_alloc(h, ptr, count); };
  const size_t B = h->B, m = h->m, R = h->R, G = h->G, V = h->V;
  A(&h->w, B * m); A(&h->pending, B * 3);
  A(&h->dev, B * G * kMaxDev); A(&h->ring, B * std::max(1, c.window_h) * kMaxDev); A(&h->running, B * kMaxDev);
  A(&h->req_ticket, 2 * B); A(&h->row_flag, B * (G + 1));
  A(&h->pushed, B); A(&h->ring_head, B); A(&h->ring_count, B); A(&h->grid_j, B);
  const size_t Dw = h->D, Rt = h->Rt;
  A(&h->qk, B * G * m * V); A(&h->q, B * G * V); A(&h->p, B * Rt * V); A(&h->scratch_q, B * V);
  A(&h->tokens, B * G); A(&h->n_accept, B); A(&h->next_token, B); A(&h->w_argmax, B);
  A(&h->cand, B * G * Dw); A(&h->acc_prim, B); A(&h->sib_tok, B);
  A(&h->chunk_mass, B * h->n_chunks); A(&h->chunk_best, B * h->n_chunks);
  A(&h->err, 1);
  A(&h->st_u_draft, B * G * Dw); A(&h->st_u_accept, B * G * Dw); A(&h->st_u_resid, B); A(&h->st_target, B * Rt * V); A(&h->st_tokens, B * G * Dw);
  if (cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking) != cudaSuccess) h->copy_stream = nullptr;
  if (cudaEventCreateWithFlags(&h->ev_round_begin, cudaEventDisableTiming) != cudaSuccess) h->ev_round_begin = nullptr;
  if (cudaEventCreateWithFlags(&h->ev_target_ready, cudaEventDisableTiming) != cudaSuccess) h->ev_target_ready = nullptr;
  cudaGetLastError();                               // (without them tabed_round_host copies on the caller's stream)
  if (h->has_drafter) {
    h->L = c.n_layers; h->d = c.d_model; h->F = c.d_ffn; h->H = c.n_heads; h->Hkv = c.n_kv_heads;
    h->hd = c.d_model / c.n_heads; h->cap = c.kv_capacity; h->esz = c.dtype == TABED_DTYPE_FP32 ? 4 : 2;
    h->qkv_w = (h->H + 2 * h->Hkv) * h->hd;
    while (h->ns > 1 && (size_t)h->ns * std::max(h->d, h->F) * sizeof(float) > 200u * 1024u) {
      const int opts[] = {1, 2, 3, 4, 6, 8};
      int lower = 1;
      for (int o : opts) if (o < h->ns) lower = o;
      h->ns = lower;
    }
    { const int shortest = std::min(64, attn_bw_split_len(h->hd)); h->max_splits = (h->cap + shortest - 1) / shortest; }   // shortest attention split of any kernel
    h->embed = wts->embed; h->lm_head = wts->lm_head; h->final_norm = wts->final_norm;
    for (int l = 0; l < h->L; ++l) {
      h->wq.push_back(wts->wq[l]); h->wk.push_back(wts->wk[l]); h->wv.push_back(wts->wv[l]); h->wo.push_back(wts->wo[l]);
      h->w_gate.push_back(wts->w_gate[l]); h->w_up.push_back(wts->w_up[l]); h->w_down.push_back(wts->w_down[l]);
      h->norm1.push_back(wts->norm1[l]); h->norm2.push_back(wts->norm2[l]);
    }
    const size_t kv_elems = R * h->L * h->Hkv * (size_t)h->cap * h->hd;
    unsigned char *kcb = nullptr, *vcb = nullptr;
    A(&kcb, kv_elems * h->esz); A(&vcb, kv_elems * h->esz);
    h->kc = kcb; h->vc = vcb;
    // step buffers: 2R slots for drafting; a bf16 drafter is prefilled in chunks of kPrefillChunk positions
    // (one slot per position) through the tensor-core kernels, which needs that many
    const size_t SC = (c.dtype == TABED_DTYPE_BF16) ? std::max<size_t>(2 * R, kPrefillChunk) : 2 * R;
    h->slot_cap = (int)SC;
    A(&h->kv_len, R); A(&h->slots, SC); A(&h->last_slot, R);
    A(&h->x, SC * h->d); A(&h->qkv, SC * h->qkv_w); A(&h->attn_out, SC * h->H * h->hd); A(&h->mid, SC * h->F);
    A(&h->part_o, SC * h->H * (size_t)h->max_splits * h->hd); A(&h->part_ml, SC * h->H * (size_t)h->max_splits * 2);
    A(&h->logits_own, G * R * V);
    A(&h->attn_tickets, SC * h->Hkv);
    if (c.dtype == TABED_DTYPE_BF16 && h->hd == kAtcHd && h->H / h->Hkv <= kMaxGroup && rc == TABED_OK) {
      // TMA descriptors of the caches seen as [all rows of all (row, layer, head)][64] bf16, tiles of 128 rows, 128-byte swizzle
      typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                   const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                   CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      const unsigned long long n_rows = (unsigned long long)R * h->L * h->Hkv * (unsigned long long)h->cap;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess && fn &&
          qres == cudaDriverEntryPointSuccess && n_rows < (1ull << 31)) {
        const cuuint64_t dims[2] = {(cuuint64_t)kAtcHd, (cuuint64_t)n_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)kAtcHd * 2};
        const cuuint32_t box[2] = {(cuuint32_t)kAtcHd, (cuuint32_t)kAtcSplit};
        const cuuint32_t estr[2] = {1, 1};
        EncodeFn enc = reinterpret_cast<EncodeFn>(fn);
        const CUresult r1 = enc(&h->tm_k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, h->kc, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        const CUresult r2 = enc(&h->tm_v, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, h->vc, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        h->atc_ok = (r1 == CUDA_SUCCESS && r2 == CUDA_SUCCESS);
      } else {
        cudaGetLastError();
      }
    }
    A(&h->rope_cos, (size_t)h->cap * (h->hd / 2)); A(&h->rope_sin, (size_t)h->cap * (h->hd / 2));
    if (rc == TABED_OK) {
      const int half = h->hd / 2;
      std::vector<float> hc((size_t)h->cap * half), hs((size_t)h->cap * half);
      for (int i = 0; i < half; ++i) {
        const double inv = pow((double)c.rope_theta, -2.0 * i / h->hd);
        for (int pos = 0; pos < h->cap; ++pos) {
          const double ang = pos * inv;
          hc[(size_t)pos * half + i] = (float)cos(ang);
          hs[(size_t)pos * half + i] = (float)sin(ang);
        }
      }
      if (cudaMemcpyAsync(h->rope_cos, hc.data(), hc.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
          cudaMemcpyAsync(h->rope_sin, hs.data(), hs.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
          cudaStreamSynchronize(h->stream) != cudaSuccess)
        rc = TABED_ERR_CUDA;
    }
    h->len_ub.assign(R, 0);
    if (rc == TABED_OK) rc = setup_persistent(h);
    if (rc == TABED_OK) rc = setup_tc(h);
  }
  if (rc == TABED_OK) {
    // equal weights before any history; one pending slot per request; grid j* undefined
    std::vector<float> w0(B * m, 1.0f / (float)m);
    std::vector<int> pend(B * 3, 0), gj(B, -1);
    for (size_t b = 0; b < B; ++b) pend[b * 3] = 1;
    if (cudaMemcpyAsync(h->w, w0.data(), w0.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaMemcpyAsync(h->pending, pend.data(), pend.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaMemcpyAsync(h->grid_j, gj.data(), gj.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess)
      rc = TABED_ERR_CUDA;
  }
  h->pend_cnt.assign(B, 1); h->pend_known = true;
  if (rc != TABED_OK) { tabed_destroy(h); cudaGetLastError(); return rc; }
  *out = h;
  return TABED_OK;
}

void tabed_destroy(tabed_handle* h) {
  if (!h) return;
  DeviceGuard guard(h->cfg.device);
  cudaStreamSynchronize(h->stream);
  for (void* ptr : h->allocs) cudaFree(ptr);
  for (cudaEvent_t e : h->prof_events) cudaEventDestroy(e);
  if (h->copy_stream) { cudaStreamSynchronize(h->copy_stream); cudaStreamDestroy(h->copy_stream); }
  if (h->ev_round_begin) cudaEventDestroy(h->ev_round_begin);
  if (h->ev_target_ready) cudaEventDestroy(h->ev_target_ready);
  cudaGetLastError();
  delete h;
}

int64_t tabed_launch_count(const tabed_handle* h) { return h ? h->launches : 0; }

int tabed_load_prefix_kv(tabed_handle* h, int32_t row, const void* k, const void* v, int32_t len) {
  if (!h || !k || !v) return TABED_ERR_NULL_PTR;
  if (!h->has_drafter || h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  if (row < 0 || row >= h->R || len < 1 || len > h->cap) return TABED_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  const size_t row_elems = (size_t)h->L * h->Hkv * h->cap * h->hd;
  const size_t width = (size_t)len * h->hd * h->esz, dpitch = (size_t)h->cap * h->hd * h->esz;
  unsigned char* kd = reinterpret_cast<unsigned char*>(h->kc) + row * row_elems * h->esz;
  unsigned char* vd = reinterpret_cast<unsigned char*>(h->vc) + row * row_elems * h->esz;
  if (cudaMemcpy2DAsync(kd, dpitch, k, width, width, (size_t)h->L * h->Hkv, cudaMemcpyDeviceToDevice, h->stream) != cudaSuccess ||
      cudaMemcpy2DAsync(vd, dpitch, v, width, width, (size_t)h->L * h->Hkv, cudaMemcpyDeviceToDevice, h->stream) != cudaSuccess ||
      cudaMemcpyAsync(h->kv_len + row, &len, sizeof(int), cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)   // &len is a stack address
    return TABED_ERR_CUDA;
  h->len_ub[row] = len;
  return TABED_OK;
}

static int prefill_common(tabed_handle* h, int32_t row, const int32_t* tokens, const float* embeds, int32_t len) {
  if (!h || (!tokens && !embeds)) return TABED_ERR_NULL_PTR;
  if (!h->has_drafter || h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  if (row < 0 || row >= h->R || len < 1) return TABED_ERR_INVALID_ARG;
  if (h->len_ub[row] + len > h->cap) return TABED_ERR_KV_OVERFLOW;
  DeviceGuard guard(h->cfg.device);
  if (h->tc_ok && h->path_sel != TABED_PATH_PER_OP) {
    // chunks of positions as slots of one weight pass: the projections are dense contractions (tcgen05), every
    // slot attends over the row's cache up to its own position (all K, V of the chunk are appended first)
    for (int t = 0; t < len; t += kPrefillChunk) {
      const int n = std::min(kPrefillChunk, len - t);
      StepArgs sa{};
      sa.mode = STEP_PREFILL; sa.prefill_row = row; sa.prefill_off = t;
      sa.prefill_tokens = tokens; sa.prefill_embeds = embeds;
      run_step_tc(h, sa, n, h->len_ub[row] + t + n, nullptr);
    }
  } else {
    for (int t = 0; t < len; ++t) {
      StepArgs sa{};
      sa.mode = STEP_PREFILL; sa.prefill_row = row; sa.prefill_off = t;
      sa.prefill_tokens = tokens; sa.prefill_embeds = embeds;
      run_step(h, sa, 1, h->len_ub[row] + t + 1, nullptr);
    }
  }
  TABED_LAUNCH(h, k_advance_len, (h->R + 127) / 128, 128, 0, h->kv_len, h->R, row, len);
  h->len_ub[row] += len;
  return check_cuda();
}

int tabed_prefill_tokens(tabed_handle* h, int32_t row, const int32_t* tokens, int32_t len) {
  return prefill_common(h, row, tokens, nullptr, len);
}
int tabed_prefill_embeds(tabed_handle* h, int32_t row, const float* embeds, int32_t len) {
  return prefill_common(h, row, nullptr, embeds, len);
}

int tabed_pool_embeds(tabed_handle* h, const float* in, int32_t grid_h, int32_t grid_w, int32_t d, float* out) {
  if (!h || !in || !out) return TABED_ERR_NULL_PTR;
  if (grid_h < 2 || grid_w < 2 || (grid_h & 1) || (grid_w & 1) || d < 1 || in == out) return TABED_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  TABED_LAUNCH(h, k_pool2x2, (grid_h / 2) * (grid_w / 2), 256, 0, in, grid_w, d, out);
  return check_cuda();
}

int tabed_set_pending(tabed_handle* h, const int32_t* tok, const int32_t* cnt) {
  if (!h || !tok || !cnt) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  std::vector<int> ht(h->B * 2), hc(h->B), pend(h->B * 3);
  if (cudaMemcpyAsync(ht.data(), tok, ht.size() * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaMemcpyAsync(hc.data(), cnt, hc.size() * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return TABED_ERR_CUDA;
  for (int b = 0; b < h->B; ++b) {
    if (hc[b] < 1 || hc[b] > 2) return TABED_ERR_INVALID_ARG;
    for (int j = 0; j < hc[b]; ++j) if (ht[b * 2 + j] < 0 || ht[b * 2 + j] >= h->V) return TABED_ERR_INVALID_ARG;
    pend[b * 3] = hc[b]; pend[b * 3 + 1] = ht[b * 2]; pend[b * 3 + 2] = hc[b] == 2 ? ht[b * 2 + 1] : 0;
  }
  if (cudaMemcpyAsync(h->pending, pend.data(), pend.size() * 4, cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return TABED_ERR_CUDA;
  h->pend_cnt = hc; h->pend_known = true;
  return TABED_OK;
}

int tabed_decode_step(tabed_handle* h, const int32_t* tok, float* out_logits) {
  if (!h || !tok) return TABED_ERR_NULL_PTR;
  if (!h->has_drafter || h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  if (max_len_ub(h) + 1 > h->cap) return TABED_ERR_KV_OVERFLOW;
  DeviceGuard guard(h->cfg.device);
  StepArgs sa{};
  sa.mode = STEP_FREE; sa.tokens = tok;
  if (use_tc(h)) run_step_tc(h, sa, h->R, max_len_ub(h) + 1, out_logits);
  else run_step(h, sa, h->R, max_len_ub(h) + 1, out_logits);
  TABED_LAUNCH(h, k_advance_len, (h->R + 127) / 128, 128, 0, h->kv_len, h->R, -1, 1);
  for (int& v : h->len_ub) v += 1;
  return check_cuda();
}

int tabed_ensemble_step(tabed_handle* h, const float* logits, const float* w, const float* u, int32_t* y,
                        float* q, float* qk) {
  if (!h || !logits || !u || !y) return TABED_ERR_NULL_PTR;
  DeviceGuard guard(h->cfg.device);
  run_ensemble(h, logits, w ? w : h->w, u, 1, y, 1, nullptr, 0, qk, (long long)h->m * h->V,
               q ? q : h->scratch_q, (long long)h->V);
  return check_cuda();
}

static int draft_common(tabed_handle* h, const float* ext_logits, const float* u_draft, int32_t* out_tokens,
                        float* out_q) {
  if (!h || !u_draft || !out_tokens) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  const bool fwd = ext_logits == nullptr;
  if (fwd && !h->has_drafter) return TABED_ERR_BAD_STATE;
  if (fwd && max_len_ub(h) + 2 + h->G - 1 > h->cap) return TABED_ERR_KV_OVERFLOW;
  DeviceGuard guard(h->cfg.device);
  const long long RV = (long long)h->R * h->V, GV = (long long)h->G * h->V;
  if (fwd && h->persist_ok && (h->path_sel == TABED_PATH_AUTO || h->path_sel == TABED_PATH_PERSISTENT)) {
    // the whole round (gamma decoder steps, each with its ensemble + draw) in one cooperative launch
    {
      ProfScope ps(h, TABED_PROF_DRAFT_ROUND);
      const int rc = launch_persistent_round(h, u_draft, out_tokens, max_len_ub(h) + 2 + h->G - 1);
      if (rc != TABED_OK) { cudaGetLastError(); return rc; }
    }
    if (out_q && cudaMemcpyAsync(out_q, h->q, sizeof(float) * h->B * GV, cudaMemcpyDeviceToDevice, h->stream) != cudaSuccess)
      return TABED_ERR_CUDA;
    h->phase = PH_DRAFTED;
    h->round_has_forward = true;
    h->cand_is_tokens = true;
    return check_cuda();
  }
  for (int i = 0; i < h->G; ++i) {
    const float* lg;
    if (fwd) {
      StepArgs sa{};
      sa.mode = (i == 0) ? STEP_ROUND_FIRST : STEP_ROUND_NEXT; sa.step = i; sa.tokens = h->tokens;
      float* own = h->logits_own + i * RV;
      if (use_tc(h)) run_step_tc(h, sa, i == 0 ? 2 * h->R : h->R, max_len_ub(h) + 2 + i, own);
      else run_step(h, sa, i == 0 ? 2 * h->R : h->R, max_len_ub(h) + 2 + i, own);
      lg = h->logits_override ? h->logits_override + i * RV : own;
    } else {
      lg = ext_logits + i * RV;
    }
    run_ensemble(h, lg, h->w, u_draft + i * h->D, h->G * h->D, h->tokens + i, h->G, out_tokens + i * h->D, h->G * h->D,
                 h->qk + (long long)i * h->m * h->V, GV * h->m, h->q + (long long)i * h->V, GV,
                 h->D, h->cand + i * h->D, h->G * h->D);
  }
  if (out_q && cudaMemcpyAsync(out_q, h->q, sizeof(float) * h->B * GV, cudaMemcpyDeviceToDevice, h->stream) != cudaSuccess)
    return TABED_ERR_CUDA;
  h->phase = PH_DRAFTED;
  h->round_has_forward = fwd;
  h->cand_is_tokens = false;
  return check_cuda();
}

int tabed_draft_round(tabed_handle* h, const float* u_draft, int32_t* out_tokens, float* out_q) {
  return draft_common(h, nullptr, u_draft, out_tokens, out_q);
}

int tabed_draft_round_logits(tabed_handle* h, const float* drafter_logits, const float* u_draft,
                             int32_t* out_tokens, float* out_q) {
  if (!drafter_logits) return TABED_ERR_NULL_PTR;
  return draft_common(h, drafter_logits, u_draft, out_tokens, out_q);
}

int tabed_verify(tabed_handle* h, const float* target_logits, const float* u_accept, const float* u_resid,
                 int32_t* out_n_accept, int32_t* out_next_token) {
  if (!h || !target_logits || !u_accept || !u_resid || !out_n_accept || !out_next_token) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_DRAFTED) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  ProfScope ps(h, TABED_PROF_VERIFY);
  VerifyArgs a{};
  const int cs = pick_cluster(h, h->B * (h->G + 1), &a.slice);
  a.row_flag = h->row_flag; a.ticket = h->req_ticket;
  a.D = h->D; a.cand = h->cand_is_tokens ? h->tokens : h->cand; a.acc_prim = h->acc_prim; a.sib_tok = h->sib_tok;
  a.V = h->V; a.G = h->G; a.greedy = h->cfg.sample_mode == TABED_MODE_GREEDY;
  a.logits = target_logits; a.q = h->q; a.q_req_stride = (long long)h->G * h->V; a.tokens = h->tokens;
  a.u_accept = u_accept; a.u_resid = u_resid; a.p = h->p;
  a.n_accept = h->n_accept; a.out_n_accept = out_n_accept == h->n_accept ? nullptr : out_n_accept;
  a.next_token = h->next_token; a.out_next_token = out_next_token == h->next_token ? nullptr : out_next_token;
  a.err = h->err;
  // With many requests the per-row clusters are small; the tail (one row-wide pass after the other) then runs as a
  // launch of its own with one cluster per request, as large as the budget allows.
  int slice_tail = 0;
  const int cs_tail = pick_cluster(h, h->B, &slice_tail);
  a.tail_inline = cs_tail >= 4 * cs ? 0 : 1;
  size_t dyn = (size_t)a.slice * sizeof(float);
  if (dyn <= kReqDynSmemMax && h->req_dyn_ok) a.ebuf_pitch = a.slice; else dyn = 0;
  launch_request_clusters(h, k_verify_req, h->B * (h->G + 1), cs, a, dyn);
  if (!a.tail_inline) {
    a.slice = slice_tail; a.ebuf_pitch = 0;
    launch_request_clusters(h, k_verify_tail, h->B, cs_tail, a);
  }
  h->phase = PH_VERIFIED;
  return check_cuda();
}

int tabed_update_weights(tabed_handle* h, float* out_w, int32_t* out_w_argmax) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_VERIFIED) return TABED_ERR_BAD_STATE;
  if (h->cfg.policy == TABED_POLICY_RANDOM && !h->u_policy) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  const int tvd = h->cfg.distance == TABED_DIST_TVD;
  {
    ProfScope ps(h, TABED_PROF_UPDATE);
    UpdateArgs u{};
    // (twice the budget: the clusters of positions that were not verified - on average ~40 % - leave at once;
    // 32 requests x 5 positions: 53.5 us with clusters of 2, 42.7 with 4, 47.7 with 8)
    const int cs = pick_cluster(h, h->B * h->G, &u.slice, 2);
    u.ticket = h->req_ticket + h->B; u.Rt = h->Rt;
    u.V = h->V;
    u.grid_policy = (h->cfg.policy == TABED_POLICY_GRID_MT || h->cfg.policy == TABED_POLICY_GRID_HARD) ? 1 : 0;
    u.hard = h->cfg.policy == TABED_POLICY_GRID_HARD ? 1 : (h->cfg.policy == TABED_POLICY_ADABOOST ? 2 : 0);
    u.p = h->p; u.qk = h->qk;
    PolicyArgs& a = u.P;
    a.B = h->B; a.G = h->G; a.m = h->m; a.n_dev = h->n_dev; a.h = h->cfg.window_h; a.policy = h->cfg.policy; a.tvd = tvd;
    a.V = h->V; a.u_policy = h->u_policy;
    a.tau = h->cfg.tau; a.n_accept = h->acc_prim; a.sib_tok = h->sib_tok; a.next_token = h->next_token; a.tokens = h->tokens;
    a.dev = h->dev; a.ring = h->ring; a.ring_head = h->ring_head; a.ring_count = h->ring_count; a.pushed = h->pushed;
    a.running = h->running; a.w = h->w; a.grid_j = h->grid_j;
    a.kv_len = (h->has_drafter && h->round_has_forward) ? h->kv_len : nullptr;
    a.pending = h->pending; a.out_w = out_w; a.out_argmax = out_w_argmax;
    launch_request_clusters(h, k_update_req, h->B * h->G, cs, u);
  }
  // the host has not seen the accept counts: the bound grows by the most a round can keep (tabed_round_host and
  // tabed_sync_lengths replace it by the exact lengths)
  if (h->has_drafter && h->round_has_forward) for (int& v : h->len_ub) v = std::min(v + h->G + 1, h->cap);
  h->pend_known = false;
  h->phase = PH_IDLE;
  return check_cuda();
}

int tabed_round_host(tabed_handle* h, const float* u_draft, const float* u_accept, const float* u_resid,
                     const float* target_logits, int32_t* out_tokens, int32_t* out_n_accept,
                     int32_t* out_next_token, float* out_w, int32_t* out_w_argmax) {
  if (!h || !u_draft || !u_accept || !u_resid || !target_logits || !out_tokens || !out_n_accept || !out_next_token)
    return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE || !h->has_drafter) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  const size_t BG = (size_t)h->B * h->G * h->D;
  cudaStream_t st = h->stream;
  const size_t target_bytes = (size_t)h->B * h->Rt * h->V * 4;
  if (cudaMemcpyAsync(h->st_u_draft, u_draft, BG * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(h->st_u_accept, u_accept, BG * 4, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(h->st_u_resid, u_resid, (size_t)h->B * 4, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return TABED_ERR_CUDA;
  const bool side = h->copy_stream && h->ev_round_begin && h->ev_target_ready;
  if (side) {
    // after everything the caller's stream holds so far (the staging buffer's last reader among it), beside the drafting
    if (cudaEventRecord(h->ev_round_begin, st) != cudaSuccess || cudaStreamWaitEvent(h->copy_stream, h->ev_round_begin, 0) != cudaSuccess ||
        cudaMemcpyAsync(h->st_target, target_logits, target_bytes, cudaMemcpyHostToDevice, h->copy_stream) != cudaSuccess ||
        cudaEventRecord(h->ev_target_ready, h->copy_stream) != cudaSuccess)
      return TABED_ERR_CUDA;
  } else if (cudaMemcpyAsync(h->st_target, target_logits, target_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    return TABED_ERR_CUDA;
  }
  const std::vector<int> len_before = h->len_ub, cnt_before = h->pend_cnt;
  const bool known_before = h->pend_known;
  // outputs land in library buffers first (tokens / n_accept / next_token / w / w_argmax)
  int rc = tabed_draft_round(h, h->st_u_draft, h->st_tokens, nullptr);
  if (rc != TABED_OK) { if (side) cudaStreamSynchronize(h->copy_stream); return rc; }
  if (side && cudaStreamWaitEvent(st, h->ev_target_ready, 0) != cudaSuccess) return TABED_ERR_CUDA;
  rc = tabed_verify(h, h->st_target, h->st_u_accept, h->st_u_resid, h->n_accept, h->next_token);
  if (rc != TABED_OK) return rc;
  rc = tabed_update_weights(h, nullptr, h->w_argmax);
  if (rc != TABED_OK) return rc;
  if (cudaMemcpyAsync(out_tokens, h->st_tokens, BG * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(out_n_accept, h->n_accept, (size_t)h->B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(out_next_token, h->next_token, (size_t)h->B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      (out_w && cudaMemcpyAsync(out_w, h->w, (size_t)h->B * h->m * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) ||
      (out_w_argmax && cudaMemcpyAsync(out_w_argmax, h->w_argmax, (size_t)h->B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess))
    return TABED_ERR_CUDA;
  std::vector<int> h_prim(h->B), h_sib(h->B);
  if (cudaMemcpyAsync(h_prim.data(), h->acc_prim, (size_t)h->B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemcpyAsync(h_sib.data(), h->sib_tok, (size_t)h->B * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TABED_ERR_CUDA;
  // the device-side error word comes back with the results (this call synchronises anyway)
  int bits = 0;
  rc = read_clear_device_error(h->err, st, &bits);
  if (rc != TABED_OK) return rc;
  if (bits) { h->pend_known = false; return map_device_error(bits); }
  if (known_before) {
    // exact lengths: a row keeps its pending token(s) and the accepted drafts that were fed
    for (int b = 0; b < h->B; ++b) {
      const int a = h_prim[b], keep = cnt_before[b] + std::min(a, h->G - 1);       // accepted tokens of the primary chain
      for (int k = 0; k < h->m; ++k) h->len_ub[b * h->m + k] = std::min(len_before[b * h->m + k] + keep, h->cap);
      h->pend_cnt[b] = (a >= h->G || h_sib[b] >= 0) ? 2 : 1;
    }
    h->pend_known = true;
  }
  return TABED_OK;
}

namespace {
// One CTA polls a flagged word for an epoch that nobody writes: the bounded wait runs out, the error bit is set
// and the kernel returns.
__global__ void __launch_bounds__(kPT) k_wait_probe(const uint2* word, int* err) {
  __shared__ PShared S;
  if (threadIdx.x == 0) S.dead = 0;
  __syncthreads();
  if (threadIdx.x == 0) ll_wait1(word, 0xFFFFFFFFu, S, err);
  __syncthreads();
}
}  // namespace

int tabed_debug_barrier_timeout(tabed_handle* h) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (!h->persist_ok) return TABED_ERR_UNSUPPORTED;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  k_wait_probe<<<1, kPT, 0, h->stream>>>(h->ll_probe, h->err);
  h->launches++;
  return tabed_last_device_error(h);
}

int tabed_set_policy_uniforms(tabed_handle* h, const float* u_policy) {
  if (!h) return TABED_ERR_NULL_PTR;
  h->u_policy = u_policy;
  return TABED_OK;
}

int tabed_last_device_error(tabed_handle* h) {
  if (!h) return TABED_ERR_NULL_PTR;
  DeviceGuard guard(h->cfg.device);
  int bits = 0;
  const int rc = read_clear_device_error(h->err, h->stream, &bits);
  return rc != TABED_OK ? rc : map_device_error(bits);
}

int tabed_sync_lengths(tabed_handle* h) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  DeviceGuard guard(h->cfg.device);
  std::vector<int> lens(h->has_drafter ? h->R : 0), pend((size_t)h->B * 3);
  if ((h->has_drafter && cudaMemcpyAsync(lens.data(), h->kv_len, lens.size() * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) ||
      cudaMemcpyAsync(pend.data(), h->pending, pend.size() * 4, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess) {
    cudaGetLastError();
    return TABED_ERR_CUDA;
  }
  for (size_t r = 0; r < lens.size(); ++r) h->len_ub[r] = lens[r];
  for (int b = 0; b < h->B; ++b) h->pend_cnt[b] = pend[(size_t)b * 3];
  h->pend_known = true;
  return TABED_OK;
}

int tabed_profile_begin(tabed_handle* h, int32_t kernel_class) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (kernel_class < 0 || kernel_class > TABED_PROF_DRAFT_ROUND) return TABED_ERR_INVALID_ARG;
  h->prof_class = kernel_class;
  h->prof_used = 0;
  return TABED_OK;
}

int tabed_profile_end(tabed_handle* h, double* total_ms, int64_t* n_intervals) {
  if (!h || !total_ms || !n_intervals) return TABED_ERR_NULL_PTR;
  DeviceGuard guard(h->cfg.device);
  h->prof_class = -1;
  if (cudaStreamSynchronize(h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  double tot = 0.0;
  const size_t pairs = h->prof_used / 2;
  for (size_t i = 0; i < pairs; ++i) {
    float ms = 0.0f;
    if (cudaEventElapsedTime(&ms, h->prof_events[2 * i], h->prof_events[2 * i + 1]) != cudaSuccess) return TABED_ERR_CUDA;
    tot += ms;
  }
  *total_ms = tot; *n_intervals = (int64_t)pairs;
  h->prof_used = 0;
  return TABED_OK;
}

int tabed_debug_override_logits(tabed_handle* h, const float* drafter_logits) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  h->logits_override = drafter_logits;
  return TABED_OK;
}

int tabed_select_path(tabed_handle* h, int32_t path) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (path < TABED_PATH_AUTO || path > TABED_PATH_TENSOR_CORE) return TABED_ERR_INVALID_ARG;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  if (path == TABED_PATH_PERSISTENT && !h->persist_ok) return TABED_ERR_UNSUPPORTED;
  if (path == TABED_PATH_TENSOR_CORE && !h->tc_ok) return TABED_ERR_UNSUPPORTED;
  h->path_sel = path;
  return TABED_OK;
}

int tabed_current_path(const tabed_handle* h) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (h->path_sel == TABED_PATH_PER_OP) return TABED_PATH_PER_OP;
  if (h->path_sel == TABED_PATH_TENSOR_CORE) return TABED_PATH_TENSOR_CORE;
  if (h->path_sel == TABED_PATH_PERSISTENT) return TABED_PATH_PERSISTENT;
  return h->persist_ok ? TABED_PATH_PERSISTENT : (h->tc_auto ? TABED_PATH_TENSOR_CORE : TABED_PATH_PER_OP);
}

int tabed_debug_trace(tabed_handle* h, int32_t on) {
  if (!h) return TABED_ERR_NULL_PTR;
  if (!h->persist_ok) return TABED_ERR_UNSUPPORTED;
  h->trace_on = on != 0;
  h->trace_cta = on > 0 ? on - 1 : 0;
  return TABED_OK;
}

int tabed_debug_view(tabed_handle* h, int32_t what, void** dev_ptr, size_t* bytes) {
  if (!h || !dev_ptr || !bytes) return TABED_ERR_NULL_PTR;
  const size_t B = h->B, m = h->m, G = h->G, V = h->V, R = h->R;
  switch (what) {
    case TABED_VIEW_QK: *dev_ptr = h->qk; *bytes = B * G * m * V * 4; break;
    case TABED_VIEW_Q: *dev_ptr = h->q; *bytes = B * G * V * 4; break;
    case TABED_VIEW_P: *dev_ptr = h->p; *bytes = B * (size_t)h->Rt * V * 4; break;
    case TABED_VIEW_ACC_PRIMARY: *dev_ptr = h->acc_prim; *bytes = B * 4; break;
    case TABED_VIEW_SIBLING: *dev_ptr = h->sib_tok; *bytes = B * 4; break;
    case TABED_VIEW_LOGITS: if (!h->has_drafter) return TABED_ERR_BAD_STATE; *dev_ptr = h->logits_own; *bytes = G * R * V * 4; break;
    case TABED_VIEW_KV_LEN: if (!h->has_drafter) return TABED_ERR_BAD_STATE; *dev_ptr = h->kv_len; *bytes = R * 4; break;
    case TABED_VIEW_WEIGHTS: *dev_ptr = h->w; *bytes = B * m * 4; break;
    case TABED_VIEW_WINDOW_SUM: *dev_ptr = h->running; *bytes = B * kMaxDev * 8; break;
    case TABED_VIEW_PENDING: *dev_ptr = h->pending; *bytes = B * 3 * 4; break;
    case TABED_VIEW_GRID_J: *dev_ptr = h->grid_j; *bytes = B * 4; break;
    case TABED_VIEW_ERROR_FLAG: *dev_ptr = h->err; *bytes = 4; break;
    case TABED_VIEW_TRACE:
      if (!h->persist_ok) return TABED_ERR_BAD_STATE;
      *dev_ptr = h->trace; *bytes = (size_t)h->G * h->trace_stride * kTraceRec * 8; break;
    default: return TABED_ERR_INVALID_ARG;
  }
  return TABED_OK;
}

// snapshot layout: header {magic, B, m, h, has_kv, R} then the arrays in a fixed order
struct Snap { void* ptr; size_t bytes; };
static std::vector<Snap> snap_parts(tabed_handle* h) {
  const size_t B = h->B, hh = std::max(1, h->cfg.window_h);
  std::vector<Snap> v = {
      {h->w, B * h->m * 4}, {h->pending, B * 3 * 4}, {h->ring, B * hh * kMaxDev * 8}, {h->running, B * kMaxDev * 8},
      {h->pushed, B * 8}, {h->ring_head, B * 4}, {h->ring_count, B * 4}, {h->grid_j, B * 4}};
  if (h->has_drafter) v.push_back({h->kv_len, (size_t)h->R * 4});
  return v;
}

int tabed_state_export(tabed_handle* h, void* host, size_t* bytes) {
  if (!h || !bytes) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  const auto parts = snap_parts(h);
  size_t total = 6 * sizeof(int32_t);
  for (const auto& s : parts) total += s.bytes;
  if (!host) { *bytes = total; return TABED_OK; }
  if (*bytes < total) return TABED_ERR_INVALID_ARG;
  DeviceGuard guard(h->cfg.device);
  int32_t hdr[6] = {0x7ABED, h->B, h->m, h->cfg.window_h, h->has_drafter ? 1 : 0, h->R};
  unsigned char* o = reinterpret_cast<unsigned char*>(host);
  memcpy(o, hdr, sizeof(hdr)); o += sizeof(hdr);
  for (const auto& s : parts) {
    if (cudaMemcpyAsync(o, s.ptr, s.bytes, cudaMemcpyDeviceToHost, h->stream) != cudaSuccess) return TABED_ERR_CUDA;
    o += s.bytes;
  }
  if (cudaStreamSynchronize(h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  if (h->has_drafter) {
    const int32_t* lens = reinterpret_cast<const int32_t*>(o - (size_t)h->R * 4);
    for (int r = 0; r < h->R; ++r) h->len_ub[r] = lens[r];      // tighten the host-side bound
  }
  *bytes = total;
  return TABED_OK;
}

int tabed_state_import(tabed_handle* h, const void* host, size_t bytes) {
  if (!h || !host) return TABED_ERR_NULL_PTR;
  if (h->phase != PH_IDLE) return TABED_ERR_BAD_STATE;
  const auto parts = snap_parts(h);
  size_t total = 6 * sizeof(int32_t);
  for (const auto& s : parts) total += s.bytes;
  if (bytes != total) return TABED_ERR_INVALID_ARG;
  const unsigned char* in = reinterpret_cast<const unsigned char*>(host);
  int32_t hdr[6];
  memcpy(hdr, in, sizeof(hdr)); in += sizeof(hdr);
  if (hdr[0] != 0x7ABED || hdr[1] != h->B || hdr[2] != h->m || hdr[3] != h->cfg.window_h ||
      hdr[4] != (h->has_drafter ? 1 : 0) || hdr[5] != h->R)
    return TABED_ERR_INVALID_ARG;
  {
    // every field that indexes memory on the device is range-checked on the host copy first: a stale or corrupt
    // snapshot is rejected without touching the device state
    const size_t B = h->B, hh = std::max(1, h->cfg.window_h);
    const unsigned char* q = in;
    q += B * h->m * 4;                                                   // w
    const int32_t* pend = reinterpret_cast<const int32_t*>(q); q += B * 3 * 4;
    q += B * hh * kMaxDev * 8 + B * kMaxDev * 8;                         // ring, running sums
    const unsigned char* pushed_raw = q; q += B * 8;                     // (64-bit fields may sit at any 4-byte offset: copied out)
    const int32_t* ring_head = reinterpret_cast<const int32_t*>(q); q += B * 4;
    const int32_t* ring_count = reinterpret_cast<const int32_t*>(q); q += B * 4;
    const int32_t* grid_j = reinterpret_cast<const int32_t*>(q); q += B * 4;
    for (size_t b = 0; b < B; ++b) {
      const int cnt = pend[b * 3];
      if (cnt < 1 || cnt > 2) return TABED_ERR_INVALID_ARG;
      for (int j = 0; j < cnt; ++j) if (pend[b * 3 + 1 + j] < 0 || pend[b * 3 + 1 + j] >= h->V) return TABED_ERR_INVALID_ARG;
      long long pushed_b;
      memcpy(&pushed_b, pushed_raw + b * 8, 8);
      if (pushed_b < 0 || ring_head[b] < 0 || ring_head[b] >= (int)hh || ring_count[b] < 0 || ring_count[b] > h->cfg.window_h ||
          grid_j[b] < -1 || grid_j[b] >= kGridCand)
        return TABED_ERR_INVALID_ARG;
    }
    if (h->has_drafter) {
      const int32_t* lens = reinterpret_cast<const int32_t*>(q);
      for (int r = 0; r < h->R; ++r) if (lens[r] < 0 || lens[r] > h->cap) return TABED_ERR_INVALID_ARG;
    }
  }
  DeviceGuard guard(h->cfg.device);
  for (const auto& s : parts) {
    if (cudaMemcpyAsync(s.ptr, in, s.bytes, cudaMemcpyHostToDevice, h->stream) != cudaSuccess) return TABED_ERR_CUDA;
    in += s.bytes;
  }
  if (cudaStreamSynchronize(h->stream) != cudaSuccess) return TABED_ERR_CUDA;
  if (h->has_drafter) {
    const int32_t* lens = reinterpret_cast<const int32_t*>(in - (size_t)h->R * 4);
    for (int r = 0; r < h->R; ++r) h->len_ub[r] = lens[r];
  }
  {
    const int32_t* pend = reinterpret_cast<const int32_t*>(reinterpret_cast<const unsigned char*>(host) + 6 * sizeof(int32_t) + (size_t)h->B * h->m * 4);
    for (int b = 0; b < h->B; ++b) h->pend_cnt[b] = pend[(size_t)b * 3];
    h->pend_known = true;
  }
  return TABED_OK;
}

// -------------------------------------------------------------------------------------------------
// Stand-alone run of the tensor-core projection (packing + k_gemm_tc + split-K sum) on caller data.
// -------------------------------------------------------------------------------------------------
namespace {
__global__ void k_sum_partials(const float* __restrict__ part, int ks, size_t elems, float* __restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= elems) return;
  float v = 0.0f;
  for (int k = 0; k < ks; ++k) v += part[(size_t)k * elems + i];
  out[i] = v;
}
}  // namespace

int tabed_debug_gemm_tc(const void* w, const float* act, int32_t rows, int32_t K, int32_t n, int32_t ks, float* out,
                        int32_t device, void* stream) {
  if (!w || !act || !out) return TABED_ERR_NULL_PTR;
  if (rows < 1 || K < 8 || (K % 8) || n < 1 || n > kTcMaxN || ks < 1 || device < 0) return TABED_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return TABED_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int m_tiles = (rows + kTcM - 1) / kTcM, k_chunks = (K + kTcKC - 1) / kTcKC, n_pad = (n + 15) / 16 * 16;
  if (ks > k_chunks) ks = k_chunks;
  const int cps = (k_chunks + ks - 1) / ks;
  unsigned char *a_p = nullptr, *b_p = nullptr; float* part = nullptr; int* err = nullptr;
  int rc = TABED_OK;
  const size_t smem = (size_t)tc_stages(n_pad) * (tc_block_bytes(kTcM) + tc_block_bytes(n_pad)) + 1024;
  if (cudaMalloc(&a_p, (size_t)m_tiles * k_chunks * tc_block_bytes(kTcM)) != cudaSuccess ||
      cudaMalloc(&b_p, (size_t)k_chunks * tc_block_bytes(n_pad)) != cudaSuccess ||
      cudaMalloc(&part, (size_t)ks * n * rows * sizeof(float)) != cudaSuccess || cudaMalloc(&err, sizeof(int)) != cudaSuccess ||
      cudaMemsetAsync(err, 0, sizeof(int), st) != cudaSuccess ||
      cudaFuncSetAttribute(k_gemm_tc, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    rc = TABED_ERR_CUDA;
  if (rc == TABED_OK) {
    k_pack_tc<<<dim3(k_chunks, m_tiles), 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16*>(w), rows, nullptr, 0, nullptr, 0, K, k_chunks, a_p);
    k_prep_act<<<k_chunks, 256, 0, st>>>(act, K, n, n_pad, K, nullptr, nullptr, b_p);
    TcGemmArgs G{};
    G.a_packed = a_p; G.b_packed = b_p; G.partial = part; G.slab = (size_t)n * rows; G.rows_total = rows; G.rows_valid = rows; G.n_pad = n_pad; G.n_slots = n;
    G.k_chunks = k_chunks; G.ks = ks; G.cps = cps; G.err = err;
    G.kc = kTcKC; G.n_stages = tc_stages(n_pad);
    k_gemm_tc<<<m_tiles * ks, kTcThreads, smem, st>>>(G);
    const size_t elems = (size_t)n * rows;
    k_sum_partials<<<(unsigned)((elems + 255) / 256), 256, 0, st>>>(part, ks, elems, out);
    int herr = 0;
    if (cudaMemcpyAsync(&herr, err, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess ||
        cudaGetLastError() != cudaSuccess)
      rc = TABED_ERR_CUDA;
    else if (herr) rc = TABED_ERR_TIMEOUT;
  }
  cudaFree(a_p); cudaFree(b_p); cudaFree(part); cudaFree(err);
  cudaGetLastError();
  return rc;
}

// -------------------------------------------------------------------------------------------------
// Allocation-free ensemble step.
//
// Scratch of the softmax / mix / draw kernels (row maxima, row sums, per-chunk masses and bests,
// an error word) lives in this file-scope device array instead of a buffer from tabed_init.  Every
// GPU that loads the library holds these 144 KB until the process exits.  In host code the name
// below is only a stand-in: its device address is fetched per device with cudaGetSymbolAddress.
// -------------------------------------------------------------------------------------------------
namespace {
constexpr size_t kStaticRowMaxOff = 0;                                                        // uint32 [MAX_ROWS]
constexpr size_t kStaticRowSumOff = kStaticRowMaxOff + 4 * (size_t)TABED_STATIC_MAX_ROWS;     // uint64 [MAX_ROWS]
constexpr size_t kStaticMassOff = kStaticRowSumOff + 8 * (size_t)TABED_STATIC_MAX_ROWS;       // uint64 [MAX_CHUNKS]
constexpr size_t kStaticBestOff = kStaticMassOff + 8 * (size_t)TABED_STATIC_MAX_CHUNKS;       // ChunkBest [MAX_CHUNKS]
constexpr size_t kStaticErrOff = kStaticBestOff + 8 * (size_t)TABED_STATIC_MAX_CHUNKS;        // int32
constexpr size_t kStaticBytes = kStaticErrOff + 256;
static_assert(sizeof(ChunkBest) == 8, "scratch layout assumes 8-byte ChunkBest");
}  // namespace

static __device__ __align__(256) unsigned char g_tabed_static_scratch[kStaticBytes];

namespace {
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {nullptr};
}  // namespace

namespace {
// device address of the static scratch on `device` (which must be current); looked up once per device
unsigned char* static_scratch_base(int device) {
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_ptr[device]) {
    void* sym = nullptr;
    if (cudaGetSymbolAddress(&sym, g_tabed_static_scratch) != cudaSuccess || !sym) { cudaGetLastError(); return nullptr; }
    g_static_ptr[device] = reinterpret_cast<unsigned char*>(sym);
  }
  return g_static_ptr[device];
}
}  // namespace

int tabed_static_last_error(int32_t device, void* stream) {
  if (device < 0 || device >= kMaxDevices) return TABED_ERR_INVALID_ARG;
  DeviceGuard guard(device);
  if (!guard.ok) return TABED_ERR_CUDA;
  unsigned char* base = static_scratch_base(device);
  if (!base) return TABED_ERR_CUDA;
  int bits = 0;
  const int rc = read_clear_device_error(reinterpret_cast<int*>(base + kStaticErrOff), reinterpret_cast<cudaStream_t>(stream), &bits);
  return rc != TABED_OK ? rc : map_device_error(bits);
}

int tabed_ensemble_step_static(const float* logits, const float* w, const float* u, int32_t n_requests,
                               int32_t n_inputs, int32_t vocab, int32_t sample_mode, int32_t device, void* stream,
                               int32_t* y, float* q, float* qk) {
  if (!logits || !w || !u || !y || !q) return TABED_ERR_NULL_PTR;
  if (n_requests < 1 || n_inputs < 1 || n_inputs > TABED_MAX_INPUTS || vocab < 2 || sample_mode < 0 || sample_mode > 1 ||
      device < 0 || device >= kMaxDevices)
    return TABED_ERR_INVALID_ARG;
  const long long rows = (long long)n_requests * n_inputs;
  const int n_chunks = (vocab + kChunk - 1) / kChunk;
  if (rows > TABED_STATIC_MAX_ROWS || (long long)n_requests * n_chunks > TABED_STATIC_MAX_CHUNKS)
    return TABED_ERR_UNSUPPORTED;                       // beyond the fixed scratch: use a handle instead
  DeviceGuard guard(device);
  if (!guard.ok) return TABED_ERR_CUDA;
  unsigned char* base = static_scratch_base(device);    // once per device, with that device current
  if (!base) return TABED_ERR_CUDA;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  uint32_t* rowmax = reinterpret_cast<uint32_t*>(base + kStaticRowMaxOff);
  unsigned long long* rowsum = reinterpret_cast<unsigned long long*>(base + kStaticRowSumOff);
  unsigned long long* cmass = reinterpret_cast<unsigned long long*>(base + kStaticMassOff);
  ChunkBest* cbest = reinterpret_cast<ChunkBest*>(base + kStaticBestOff);
  int* err = reinterpret_cast<int*>(base + kStaticErrOff);
  // the array keeps the previous call's contents: the running maxima and sums must start at zero
  if (cudaMemsetAsync(rowmax, 0, sizeof(uint32_t) * rows, st) != cudaSuccess ||
      cudaMemsetAsync(rowsum, 0, sizeof(unsigned long long) * rows, st) != cudaSuccess)
    return TABED_ERR_CUDA;
  const int R = (int)rows, B = n_requests, V = vocab, greedy = sample_mode == TABED_MODE_GREEDY;
  const dim3 grid_rows(n_chunks, R), grid_req(n_chunks, B);
  k_rowmax<<<grid_rows, kDecThreads, 0, st>>>(logits, V, (long long)V, rowmax);
  k_expsum<<<grid_rows, kDecThreads, 0, st>>>(logits, V, (long long)V, rowmax, rowsum);
  k_mix<<<grid_req, kDecThreads, 0, st>>>(logits, V, n_inputs, w, rowmax, rowsum, qk, (long long)n_inputs * V, q,
                                          (long long)V, cmass, cbest, n_chunks, greedy);
  SelectArgs s{};
  s.V = V; s.n_chunks = n_chunks; s.G = 1; s.greedy = greedy;
  s.q = q; s.q_req_stride = V; s.u = u; s.u_stride = 1;
  s.chunk_mass = cmass; s.chunk_best = cbest;
  s.out0 = y; s.out0_stride = 1; s.out1 = nullptr; s.out1_stride = 0; s.err = err;
  k_select<0><<<B, kDecThreads, 0, st>>>(s);
  return check_cuda();
}

}  // extern "C"
