// Host side of the ADORE C ABI: the cache object, argument checks, launch sequences.
#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <initializer_list>
#include <new>
#include <vector>

#include "../../include/adore.h"
#include "attention.cuh"
#include "attention_tma.cuh"
#include "attention_split.cuh"
#include "controller.cuh"
#include "rebuild_simt.cuh"
#include "rebuild_tc.cuh"
#include "select.cuh"
#include "labels.cuh"
#include "attention_rows.cuh"

using namespace adore;

namespace {

constexpr int kMaxPrefillRows = 8192;       // controller rows per chunk during a bulk load

// ---- kernels that glue the device functions together -----------------------------------------
// One step's selection for sequence blockIdx.x. It ranks tokens 0..n-1 by the scores they already have, so it
// does not wait for the controller's score of the new token n (that score is first read at step n+1) and runs
// beside the controller kernels.
__global__ void __launch_bounds__(512, 2) select_kernel(const SelectParams sp) {
  extern __shared__ __align__(128) unsigned char smem[];
  let_next_grid_start();
  select_step(sp, smem);
}

// Keeps the new token's layer-input row (it is what a later rebuild recomputes from, and what the controller reads):
// row b of x_new goes to position n of sequence b in the token store. One CTA per sequence, 16-byte pieces.
__global__ void __launch_bounds__(256) store_row_kernel(const uint4* x_new, uint4* x_store, int row_pieces, long long seq_pieces,
                                                        long long at_pieces) {
  const uint4* src = x_new + size_t(blockIdx.x) * row_pieces;
  uint4* dst = x_store + size_t(blockIdx.x) * seq_pieces + at_pieces;
  for (int i = threadIdx.x; i < row_pieces; i += blockDim.x) dst[i] = src[i];
}

__global__ void __launch_bounds__(512) ctrl_recur_kernel(const RecurParams rp, int resident, unsigned* err) {
  extern __shared__ __align__(128) unsigned char smem[];
  if (resident) controller_tokens_resident(rp, blockIdx.x, smem, err);
  else controller_tokens(rp, blockIdx.x, reinterpret_cast<double*>(smem));
}

__global__ void __launch_bounds__(512) bulk_select_kernel(const SelectParams sp) {
  extern __shared__ __align__(128) unsigned char smem[];
  select_bulk(sp, smem);
}

// Writes the new token's key/value rows of layer 0 into the admitted slot: one warp per (b, h).
__global__ void admit_rows_kernel(unsigned char* Kc, unsigned char* Vc, const unsigned char* k_new, const unsigned char* v_new,
                                  const int* admit_slot, int H, int C, int row_bytes, unsigned* err) {
  let_next_grid_start();
  const int bh = blockIdx.x, b = bh / H, s = admit_slot[b];
  if (s < 0 || s >= C) { if (threadIdx.x == 0) set_error(err, ERRW_BOUNDS); return; }
  const size_t dst = (size_t(bh) * C + s) * row_bytes, src = size_t(bh) * row_bytes;
  for (int i = threadIdx.x; i < row_bytes / 16; i += 32) {
    reinterpret_cast<uint4*>(Kc + dst)[i] = reinterpret_cast<const uint4*>(k_new + src)[i];
    reinterpret_cast<uint4*>(Vc + dst)[i] = reinterpret_cast<const uint4*>(v_new + src)[i];
  }
}

// Cumulative attention as the tokens' value (Section 3.1, baselines 6 and 7): every attended token gains the weight its
// row received in this launch, summed over the heads in ascending order. One thread per (sequence, slot).
__global__ void add_attention_kernel(const float* weights, const int* slot_tok, int H, int C, int n_cur, int max_tokens,
                                     float* score) {
  const int b = blockIdx.x, s = blockIdx.y * blockDim.x + threadIdx.x;
  let_next_grid_start();
  wait_for_prior_grid();
  if (s > C) return;
  const int tok = s == C ? n_cur : slot_tok[size_t(b) * C + s];
  if (tok < 0) return;
  float acc = 0.f;
  for (int h = 0; h < H; ++h) acc += weights[(size_t(b) * H + h) * (C + 1) + s];
  score[size_t(b) * max_tokens + tok] += acc;
}

__global__ void fill_i32_kernel(int* p, int v, size_t n) {
  for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n; i += size_t(gridDim.x) * blockDim.x) p[i] = v;
}

int pow2_at_least(int v) {
  int p = 2;
  while (p < v) p <<= 1;
  return p;
}

}  // namespace

struct adore_cache {
  adore_config_t cfg{};
  cudaStream_t stream = nullptr;
  size_t esz = 2;
  int n = 0;                    // tokens per sequence
  int step_layer0_done = 0;     // a step is open (layer 0 ran)
  int64_t launches = 0;
  int cur = 0, attn = 0;        // slot-map buffers: target state / state the cache rows follow

  void* Kc = nullptr;
  void* Vc = nullptr;
  void* x_store = nullptr;
  double* z = nullptr;
  double* a_tab = nullptr;      // relative positions: per token the input of the controller's Tanh layer at distance 0
  double* c_vec = nullptr;      // relative positions: W1 pos_w
  float* score = nullptr;
  float* sigma = nullptr;
  int* tok_slot = nullptr;
  int* slot_tok[2] = {nullptr, nullptr};
  uint8_t* slot_role[2] = {nullptr, nullptr};
  int* admit_slot = nullptr;
  int* evicted_tok = nullptr;
  int* rebuild_tok = nullptr;
  int* rebuild_slot = nullptr;
  int* rebuild_count = nullptr;
  int* row_b = nullptr;
  int* row_tok = nullptr;
  int* row_slot = nullptr;
  int* row_total = nullptr;
  int* frow_b = nullptr;        // row table of a layer fill (all residents)
  int* frow_tok = nullptr;
  int* frow_slot = nullptr;
  int* frow_total = nullptr;
  unsigned long long* rows_accum = nullptr;
  unsigned* sel_done = nullptr;     // arrivals of a selection launch's CTAs (the last one builds the row table)
  int sms = 148;
  unsigned* err = nullptr;
  // optional per-stage timing
  bool timing = false;
  std::vector<cudaEvent_t> ev_pool;        // start/stop pairs, reused after each read-out
  size_t ev_used = 0;
  std::vector<int> ev_stage;
  double stage_ms[4] = {0, 0, 0, 0};        // attention, controller+selection, rebuild, admit (layer 0)
  int64_t stage_launches[4] = {0, 0, 0, 0};
  // optional group timing: the step's schedule is left as it is (side streams and all); three events per step mark where
  // the attention + selection group starts, where its main-stream part ends (the last layer's attention, or the new
  // token's row of a one-layer cache) and where the controller chain ends
  bool group_timing = false;
  std::vector<cudaEvent_t> grp_pool;
  size_t grp_used = 0;
  double grp_ms = 0, grp_main_ms = 0;
  int64_t grp_steps = 0;
  double* part = nullptr;
  size_t part_doubles = 0;
  int ksplit = 1;
  float* rope_cos = nullptr;
  float* rope_sin = nullptr;
  // controller parameters on the device
  float *w_ih = nullptr, *w_hh = nullptr, *b_ih = nullptr, *b_hh = nullptr, *pos_w = nullptr, *pos_b = nullptr,
        *w1 = nullptr, *b1 = nullptr, *w2 = nullptr, *b2 = nullptr;
  // side stream: the controller and the selection run beside the attention of layer 0
  cudaStream_t aux = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  // second side stream: the controller (gates, then GRU + MLP) of the new token. Its score is first needed by
  // the NEXT step's selection, so it may run on past the end of the step that launched it.
  cudaStream_t ctl = nullptr;
  cudaEvent_t ev_xrow = nullptr, ev_attn = nullptr, ev_ctrl = nullptr;   // the token's row is in the store / the attention of layer 0 is done
  cudaEvent_t ev_gather = nullptr;  // the early gather of a short list (selection stream) is done: the rebuild waits for it
  bool xrow_pending = false, gather_pending = false;   // events the main stream / the rebuild's stream has not waited for yet
  bool ctrl_pending = false;    // ev_ctrl was recorded and the main stream has not waited for it yet
  // uploads of the host-buffer entry point run on their own stream, beside the previous rebuild
  cudaStream_t copy = nullptr;
  cudaEvent_t ev_copy = nullptr;
  cudaEvent_t ev_out = nullptr;     // `out` has reached the host (host-buffer entry point that also queues the rebuild)
  bool joined = true;
  // Caches of several layers, attend-first order: the rebuild of layer l writes layer l's rows only, which nothing reads
  // before the NEXT step's attention of that layer, so it runs on a stream of its own beside the attention of the layers
  // that follow. ev_rebuilt[l] marks its end; whoever next touches layer l's rows, the row table or the gather buffer
  // waits for it.
  cudaStream_t rb = nullptr;
  cudaEvent_t ev_rb_fork = nullptr;
  cudaEvent_t ev_step_open = nullptr;   // rebuild-first order: the main stream at the end of adore_step_begin
  std::vector<cudaEvent_t> ev_rebuilt;
  std::vector<char> rb_pending;
  int rb_last = -1;             // layer of the most recent launch on `rb` that nobody has waited for yet
  std::vector<const void*> w_kv;
  TcState tc;                   // tensor-core rebuild path (tensor maps, gather buffer)
  std::vector<CUtensorMap> map_k, map_v;   // per layer: the cache as [B*H*C, dh] tiles of 64 x 64 (bf16, dh 64 or 128)
  float* w_internal = nullptr;  // [B,H,C+1] weights when the caller passes none but the scores need them
  bool rows_gathered = false;   // the gather buffer holds this step's listed rows, taken from the token store
  // staging for the host-buffer entry point
  void *h_q = nullptr, *h_k = nullptr, *h_v = nullptr, *h_x = nullptr, *h_out = nullptr;
  int* h_list = nullptr;
  int* h_count = nullptr;
  // staging of the queued host-buffer entry point: one set per layer (several layers' calls are in flight at once)
  unsigned char* hq_all = nullptr;              // [L][4][B*H*dh] elements: q, k, v, out
  void* hq_x = nullptr;
  int* hq_list = nullptr;
  int* hq_count = nullptr;
  std::vector<cudaEvent_t> ev_stage_free;       // per layer: every reader of the layer's staging set is done
  cudaStream_t d2h = nullptr;                   // `out` goes back on its own stream, beside the next layer's attention
  std::vector<void*> owned;
};

namespace {

#define CUDA_OK(expr)                                   \
  do {                                                  \
    cudaError_t e_ = (expr);                            \
    if (e_ != cudaSuccess) return cuda_fail(e_);        \
  } while (0)

// Brackets the launches made during its lifetime with a pair of events when timing is on.
struct StageScope {
  adore_cache* c;
  size_t idx = 0;
  bool on = false;
  cudaStream_t st;
  StageScope(adore_cache* cache, int stage, cudaStream_t stream = nullptr) : c(cache), st(stream ? stream : cache->stream) {
    if (!c->timing) return;
    if (c->ev_used + 2 > c->ev_pool.size()) {
      cudaEvent_t a, b;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) return;
      c->ev_pool.push_back(a);
      c->ev_pool.push_back(b);
    }
    idx = c->ev_used;
    c->ev_used += 2;
    c->ev_stage.push_back(stage);
    cudaEventRecord(c->ev_pool[idx], st);
    on = true;
  }
  ~StageScope() { if (on) cudaEventRecord(c->ev_pool[idx + 1], st); }
};

// Group timing: the idx-th event (0 start, 1 end on the main stream, 2 end of the controller chain) of the open step.
adore_status_t group_mark(adore_cache* c, int idx, cudaStream_t stream) {
  if (!c->group_timing) return ADORE_OK;
  if (idx == 0) {
    if (c->grp_used + 3 > c->grp_pool.size())
      for (int i = 0; i < 3; ++i) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess) return ADORE_ERR_CUDA;
        c->grp_pool.push_back(e);
      }
    c->grp_used += 3;
  }
  if (c->grp_used < 3) return ADORE_OK;
  return cudaEventRecord(c->grp_pool[c->grp_used - 3 + idx], stream) == cudaSuccess ? ADORE_OK : ADORE_ERR_CUDA;
}

adore_status_t cuda_fail(cudaError_t e) {
  if (e == cudaErrorMemoryAllocation) { cudaGetLastError(); return ADORE_ERR_OOM; }
  return ADORE_ERR_CUDA;
}

// Makes the main stream wait for a controller launch that is still running on its side stream.
adore_status_t join_controller(adore_cache* c) {
  if (c->ctrl_pending) {
    CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_ctrl, 0));
    c->ctrl_pending = false;
  }
  return ADORE_OK;
}

// The kernels fetch rows of q, k, v, x and the row tables' sources in 16-byte pieces: a device pointer that does not
// start on such a boundary is refused on the host (a misaligned access would fault the device).
inline bool misaligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

// Makes `stream` wait for the rebuild of `layer` if it is still running beside the main stream.
adore_status_t wait_rebuild(adore_cache* c, int layer, cudaStream_t stream) {
  if (layer >= 0 && layer < int(c->rb_pending.size()) && c->rb_pending[layer])
    CUDA_OK(cudaStreamWaitEvent(stream, c->ev_rebuilt[layer], 0));
  return ADORE_OK;
}
// Makes the main stream wait for every rebuild that runs beside it. The side stream runs them in order, so the
// event of the most recent one covers all.
adore_status_t join_rebuilds(adore_cache* c) {
  if (c->gather_pending) {        // an early gather that no rebuild on the main stream has waited for
    CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_gather, 0));
    c->gather_pending = false;
  }
  if (c->rb_last >= 0) CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_rebuilt[c->rb_last], 0));
  c->rb_last = -1;
  std::fill(c->rb_pending.begin(), c->rb_pending.end(), char(0));
  return ADORE_OK;
}

template <typename P>
adore_status_t dev_alloc(adore_cache* c, P** out, size_t bytes, bool zero) {
  void* p = nullptr;
  CUDA_OK(cudaMalloc(&p, bytes ? bytes : 16));
  c->owned.push_back(p);
  if (zero) CUDA_OK(cudaMemsetAsync(p, 0, bytes ? bytes : 16, c->stream));
  *out = static_cast<P*>(p);
  return ADORE_OK;
}

// A group of device buffers that only make sense together: either all exist afterwards (owned by the cache), or none
// does and nothing is left behind.
struct GroupItem { void** out; size_t bytes; };
adore_status_t alloc_group(adore_cache* c, std::initializer_list<GroupItem> items) {
  std::vector<void*> got;
  for (const GroupItem& it : items) {
    void* p = nullptr;
    if (cudaMalloc(&p, it.bytes ? it.bytes : 16) != cudaSuccess) {
      cudaGetLastError();
      for (void* g : got) cudaFree(g);
      return ADORE_ERR_OOM;
    }
    got.push_back(p);
  }
  size_t i = 0;
  for (const GroupItem& it : items) { *it.out = got[i]; c->owned.push_back(got[i]); ++i; }
  return ADORE_OK;
}

adore_status_t upload(adore_cache* c, float** out, const float* host, size_t count) {
  adore_status_t s = dev_alloc(c, out, count * sizeof(float), false);
  if (s != ADORE_OK) return s;
  CUDA_OK(cudaMemcpyAsync(*out, host, count * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  CUDA_OK(cudaStreamSynchronize(c->stream));   // the host buffer may be a temporary
  return ADORE_OK;
}

adore_status_t fill_i32(adore_cache* c, int* p, int v, size_t n) {
  const int blocks = int(std::min<size_t>((n + 255) / 256, 1184));
  fill_i32_kernel<<<blocks ? blocks : 1, 256, 0, c->stream>>>(p, v, n);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  return ADORE_OK;
}

// One CTA per sequence owns an SM for a latency-bound chain (GRU, MLP, sort): the more warps, the better
// the loads and barriers are hidden.
int select_threads(const adore_cache*) { return 512; }
// The step's selection runs beside the attention of layer 0. With few (batch, head) pairs that launch has 256-thread
// CTAs of 16k registers, three or four to an SM: a selection CTA of 256 threads x 64 registers still fits beside three
// of them and starts at once, one of 512 threads waits until an SM has drained (measured: 14 us later).
// (Eight warps sort or scan at most 4096 keys, 512 each: wider candidate sets keep the 512-thread CTA.)
int step_select_threads(const adore_cache* c, int P) {
  const adore_config_t& f = c->cfg;
  return f.batch * f.n_heads < 1024 && P <= 4096 ? 256 : 512;
}
size_t ctrl_smem(const adore_cache* c) {
  const int h = c->cfg.ctrl_hidden;
  return ctrl_resident_ok(h) ? ctrl_resident_smem_bytes(h) : recur_smem_bytes(h);
}

RecurParams recur_params(adore_cache* c, int rows, int tc, int ksplit, int n0) {
  RecurParams r{};
  r.part = c->part; r.ksplit = ksplit; r.rows = rows; r.tc = tc; r.h = c->cfg.ctrl_hidden;
  r.b_ih = c->b_ih; r.w_hh = c->w_hh; r.b_hh = c->b_hh; r.pos_w = c->pos_w; r.pos_b = c->pos_b;
  r.w1 = c->w1; r.b1 = c->b1; r.w2 = c->w2; r.b2 = c->b2;
  r.z = c->z; r.score = c->score; r.sigma = c->sigma; r.max_tokens = c->cfg.max_tokens; r.n0 = n0;
  r.pos_scale = double(c->cfg.pos_scale);
  r.no_recurrence = (c->cfg.flags & ADORE_FLAG_NO_RECURRENCE) ? 1 : 0;
  r.a_tab = c->a_tab;
  return r;
}

SelectParams select_params(adore_cache* c, int n, int P, int old_map, int new_map) {
  SelectParams s{};
  s.B = c->cfg.batch; s.C = c->cfg.capacity; s.m = c->cfg.capacity - c->cfg.rebuild_max; s.r_max = c->cfg.rebuild_max;
  s.n = n; s.max_tokens = c->cfg.max_tokens; s.explicit_mode = c->cfg.rebuild_mode == ADORE_REBUILD_EXPLICIT; s.P = P;
  s.slot_tok_old = c->slot_tok[old_map]; s.slot_role_old = c->slot_role[old_map];
  s.slot_tok_new = c->slot_tok[new_map]; s.slot_role_new = c->slot_role[new_map];
  s.tok_slot = c->tok_slot; s.score = c->score;
  s.admit_slot = c->admit_slot; s.evicted_tok = c->evicted_tok; s.rebuild_tok = c->rebuild_tok;
  s.rebuild_slot = c->rebuild_slot; s.rebuild_count = c->rebuild_count;
  s.err = c->err;
  return s;
}

template <typename T>
adore_status_t launch_gates(adore_cache* c, const T* x, long long seq_stride, int tc, int ksplit, cudaStream_t stream,
                            int hh_slices = 0) {
  GateParams<T> g{};
  g.hh_slices = hh_slices; g.h = c->cfg.ctrl_hidden; g.w_hh = c->w_hh; g.z = c->z;
  g.x = x; g.seq_stride = seq_stride; g.tc = tc; g.rows = c->cfg.batch * tc; g.d = c->cfg.hidden; g.G = 3 * c->cfg.ctrl_hidden;
  g.w_ih = c->w_ih; g.part = c->part; g.ksplit = ksplit;
  const int per = (c->cfg.hidden + ksplit - 1) / ksplit;
  g.kslice = ((per + kGateKInner - 1) / kGateKInner) * kGateKInner;
  static const bool narrow_only = dev_switch("ADORE_GATES_NARROW");
  if (g.rows >= kGateWideMinRows && !narrow_only) {
    dim3 grid((g.G + kGateWideG - 1) / kGateWideG, (g.rows + kGateWideR - 1) / kGateWideR, ksplit + hh_slices);
    ctrl_gates_wide_kernel<T><<<grid, kGateWideThreads, kGateWideSmem, stream>>>(g);
    ++c->launches;
    CUDA_OK(cudaGetLastError());
    return ADORE_OK;
  }
  dim3 grid((g.G + kGateTileG - 1) / kGateTileG, (g.rows + kGateTileR - 1) / kGateTileR, ksplit + hh_slices);
  ctrl_gates_kernel<T><<<grid, kGateThreads, 0, stream>>>(g);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  return ADORE_OK;
}

template <typename T>
bool launch_attention_rows(adore_cache*, int, const AttnParams<T>&, int) { return false; }

constexpr size_t kRowsSmemLimit = 226 * 1024;             // dynamic shared memory a CTA of the rows kernel may ask for

template <int DH, int KPL, int RB>
bool launch_attention_rows_as(adore_cache* c, int layer, const AttnParams<__nv_bfloat16>& p, size_t smem) {
  static bool opted = false;                                // per instantiation
  if (!opted) {
    if (cudaFuncSetAttribute(attention_rows_kernel<DH, KPL, RB>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kRowsSmemLimit)) != cudaSuccess) {
      cudaGetLastError();
      return false;
    }
    opted = true;
  }
  const dim3 grid(unsigned(c->cfg.batch * c->cfg.n_heads)), block(kRowsThreads);
  cudaError_t e = launch_dependent(attention_rows_kernel<DH, KPL, RB>, grid, block, smem, c->stream, c->map_k[layer], c->map_v[layer], p);
  ++c->launches;
  if (e != cudaSuccess) { cudaGetLastError(); return false; }
  return true;
}

template <int DH, int RB>
bool launch_attention_rows_kpl(adore_cache* c, int layer, const AttnParams<__nv_bfloat16>& p, size_t smem, int per_lane) {
  if (per_lane <= 9) return launch_attention_rows_as<DH, 9, RB>(c, layer, p, smem);
  if (per_lane <= 17) return launch_attention_rows_as<DH, 17, RB>(c, layer, p, smem);
  return launch_attention_rows_as<DH, 33, RB>(c, layer, p, smem);
}

template <>
bool launch_attention_rows<__nv_bfloat16>(adore_cache* c, int layer, const AttnParams<__nv_bfloat16>& p, int rows_q) {
  const adore_config_t& f = c->cfg;
  static const bool off = dev_switch("ADORE_ROWS_SIMT");
  const int per_lane = (f.capacity + 1 + 31) / 32;
  if (off || c->map_k.empty() || per_lane > kRowsKeysPerLaneMax) return false;
  // Rows per launch: up to 16 with two CTAs per SM; more rows go through the three-block kernel, as many per launch as
  // the logits of a pair fit in shared memory (one pass over the pair's keys and values for all of them). What is
  // left goes in further launches of the same size; the last group holds the current token's row and stores its rows.
  int group = std::min(rows_q, kRowsMaxQ);
  if (rows_q > kRowsMaxQ) {
    group = std::min(rows_q, kRowsMaxQ * kRowsMaxBlocks);
    while (group > kRowsMaxQ && rows_smem_bytes(f.capacity, f.head_dim, group) > kRowsSmemLimit) --group;
  }
  const size_t smem = rows_smem_bytes(f.capacity, f.head_dim, group);
  if (smem > (group > kRowsMaxQ ? kRowsSmemLimit : size_t(200 * 1024))) return false;
  for (int rb = 0; rb < rows_q; rb += group) {
    AttnParams<__nv_bfloat16> g = p;
    g.rows_q = std::min(group, rows_q - rb);
    g.row_base = rb;
    g.rows_total = rows_q;
    if (rb + g.rows_q < rows_q) g.admit_slot = nullptr;
    bool ok;
    if (group > kRowsMaxQ)
      ok = f.head_dim == 128 ? launch_attention_rows_kpl<128, kRowsMaxBlocks>(c, layer, g, smem, per_lane)
                             : launch_attention_rows_kpl<64, kRowsMaxBlocks>(c, layer, g, smem, per_lane);
    else
      ok = f.head_dim == 128 ? launch_attention_rows_kpl<128, 1>(c, layer, g, smem, per_lane)
                             : launch_attention_rows_kpl<64, 1>(c, layer, g, smem, per_lane);
    // a refused first launch leaves the other kernel to do all rows; a later one cannot fail where the first did not
    if (!ok) return false;
  }
  return true;
}

template <typename T>
adore_status_t launch_attention(adore_cache* c, int layer, const void* q, const void* k_new, const void* v_new,
                                void* out, float* weights, bool fused_admit, int rows_q = 1) {
  const adore_config_t& f = c->cfg;
  AttnParams<T> p{};
  const size_t layer_elems = size_t(f.batch) * f.n_heads * f.capacity * f.head_dim;
  p.q = static_cast<const T*>(q); p.k_new = static_cast<const T*>(k_new); p.v_new = static_cast<const T*>(v_new);
  p.out = static_cast<T*>(out); p.weights = weights;
  p.Kc = static_cast<T*>(c->Kc) + layer * layer_elems; p.Vc = static_cast<T*>(c->Vc) + layer * layer_elems;
  p.slot_tok = c->slot_tok[c->attn]; p.admit_slot = fused_admit ? c->admit_slot : nullptr;
  p.rows_q = rows_q; p.row_tok = c->rebuild_tok; p.r_max = f.rebuild_max; p.n_cur = c->n - 1;
  p.B = f.batch; p.H = f.n_heads; p.C = f.capacity; p.topk = f.topk;
  p.scale = float(1.0 / std::sqrt(double(f.head_dim)));
  p.err = c->err;
  const int grid = f.batch * f.n_heads * rows_q;
  StageScope scope(c, 0);
  cudaError_t e;
  // Few (b, h) pairs: a cluster of CTAs shares each of them. Not at layer 0: there the controller's
  // one-CTA-per-sequence kernel (200 KB of shared memory each) runs beside the attention and needs
  // SMs that the extra CTAs would occupy; measured at batch 1 the step got slower, not faster.
  if (rows_q > 1) {
    // up to 16 rows on bfloat16 caches: the tensor-core kernel, one pass over the pair's keys and values for all rows
    if (launch_attention_rows<T>(c, layer, p, rows_q)) return ADORE_OK;
    // otherwise the staged kernel once per row (rows of a pair adjacent in the grid, sharing the blocks through L2)
    if (!attn_tma_usable<T>(f.capacity, f.head_dim)) return ADORE_ERR_UNSUPPORTED;
    cudaError_t er = launch_attention_tma<T>(p, f.head_dim, grid, c->stream);
    ++c->launches;
    CUDA_OK(er);
    return ADORE_OK;
  }
  if (!attn_tma_usable<T>(f.capacity, f.head_dim)) return ADORE_ERR_UNSUPPORTED;
  const int split = layer == 0 ? 1 : attn_split_factor(grid, f.capacity, c->sms);
  if (split > 1) e = launch_attention_split<T>(p, f.head_dim, grid, split, c->stream);
  else e = launch_attention_tma<T>(p, f.head_dim, grid, c->stream);
  ++c->launches;
  CUDA_OK(e);
  return ADORE_OK;
}

template <typename T>
adore_status_t launch_rebuild(adore_cache* c, int layer, const void* x_table, const int* row_b, const int* row_tok,
                              const int* row_slot, const int* row_total, int m_max, bool step_table,
                              cudaStream_t stream = nullptr) {
  const adore_config_t& f = c->cfg;
  if (m_max <= 0) return ADORE_OK;
  if (!stream) stream = c->stream;
  RebuildParams<T> p{};
  const size_t layer_elems = size_t(f.batch) * f.n_heads * f.capacity * f.head_dim;
  p.x_table = static_cast<const T*>(x_table ? x_table : c->x_store); p.seq_stride = f.max_tokens; p.d = f.hidden;
  p.w_kv = static_cast<const T*>(c->w_kv[layer]);
  p.Kc = static_cast<T*>(c->Kc) + layer * layer_elems; p.Vc = static_cast<T*>(c->Vc) + layer * layer_elems;
  p.row_b = row_b; p.row_tok = row_tok; p.row_slot = row_slot; p.row_total = row_total; p.row_base = 0; p.row_limit = m_max;
  p.rope_cos = f.rope_theta != 0.f ? c->rope_cos : nullptr; p.rope_sin = f.rope_theta != 0.f ? c->rope_sin : nullptr;
  p.H = f.n_heads; p.DH = f.head_dim; p.C = f.capacity; p.N = 2 * f.n_heads * f.head_dim; p.err = c->err;
  StageScope scope(c, 2);
  if (tc_usable<T>(c->tc)) {
    // Rows gathered from the token store for this step's table serve every layer that rebuilds from the store.
    const bool from_store = step_table && x_table == nullptr && size_t(m_max) <= c->tc.a_rows;
    int launched = 0;
    // the early gather of this step's list (selection stream) writes the buffer that this launch reads or refills
    if (c->gather_pending) {
      CUDA_OK(cudaStreamWaitEvent(stream, c->ev_gather, 0));
      if (stream == c->stream) c->gather_pending = false;       // (a side stream: every rebuild of the step waits)
    }
    static const int lean_mode = dev_switch_int("ADORE_REBUILD_LEAN", 1);
    cudaError_t e = launch_rebuild_tc(c->tc, p, layer, m_max, stream, &launched, from_store && c->rows_gathered,
                                      lean_mode != 0 && stream != c->stream);
    c->launches += launched;
    c->rows_gathered = from_store;
    CUDA_OK(e);
    return ADORE_OK;
  }
  dim3 grid(p.N / kSimtTile, (m_max + kSimtTile - 1) / kSimtTile);
  rebuild_simt_kernel<T><<<grid, 256, 0, stream>>>(p);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  return ADORE_OK;
}

// Adds the weights of the attention launch that just ran (caller's buffer or the internal one) to the tokens' scores.
adore_status_t launch_add_attention(adore_cache* c, const float* weights) {
  const adore_config_t& f = c->cfg;
  StageScope scope(c, 1);
  CUDA_OK(launch_dependent(add_attention_kernel, dim3(f.batch, (f.capacity + 1 + 127) / 128), dim3(128), 0, c->stream, weights,
                           c->slot_tok[c->attn], f.n_heads, f.capacity, c->n - 1, f.max_tokens, c->score));
  ++c->launches;
  return ADORE_OK;
}

// Relative positions: tokens 0 .. n-1 scored as seen from token n. Needs the controller launches of all of them.
adore_status_t launch_rescore(adore_cache* c, int n, cudaStream_t stream) {
  if (!c->a_tab || n < 1) return ADORE_OK;
  RescoreParams p{};
  p.a_tab = c->a_tab; p.c_vec = c->c_vec; p.w2 = c->w2; p.b2 = c->b2; p.score = c->score; p.sigma = c->sigma;
  p.h = c->cfg.ctrl_hidden; p.max_tokens = c->cfg.max_tokens; p.n = n; p.pos_scale = double(c->cfg.pos_scale);
  dim3 grid((n + kRescoreTokens - 1) / kRescoreTokens, c->cfg.batch);
  ctrl_rescore_kernel<<<grid, kRescoreThreads, 0, stream>>>(p);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  return ADORE_OK;
}

adore_status_t launch_row_table(adore_cache* c, bool count_rows, cudaStream_t stream) {
  const adore_config_t& f = c->cfg;
  if (f.rebuild_max == 0) return ADORE_OK;          // row_total stays 0
  CUDA_OK(launch_dependent(row_table_kernel, dim3(f.batch), dim3(128), 0, stream, c->rebuild_tok, c->rebuild_slot,
                           c->rebuild_count, f.batch, f.rebuild_max, c->row_b, c->row_tok, c->row_slot, c->row_total,
                           count_rows ? c->rows_accum : nullptr));
  ++c->launches;
  return ADORE_OK;
}

adore_status_t fill_layer_impl(adore_cache* c, int layer, const void* x_table) {
  const adore_config_t& f = c->cfg;
  resident_rows_kernel<<<1, 1024, 0, c->stream>>>(c->slot_tok[c->cur], f.batch, f.capacity, c->frow_b, c->frow_tok,
                                                  c->frow_slot, c->frow_total);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  if (f.dtype == ADORE_F32)
    return launch_rebuild<float>(c, layer, x_table, c->frow_b, c->frow_tok, c->frow_slot, c->frow_total, f.batch * f.capacity, false);
  return launch_rebuild<__nv_bfloat16>(c, layer, x_table, c->frow_b, c->frow_tok, c->frow_slot, c->frow_total,
                                       f.batch * f.capacity, false);
}

adore_status_t check_config(const adore_config_t* f) {
  if (f->struct_size != sizeof(adore_config_t)) return ADORE_ERR_INVALID_ARG;
  if (f->batch < 1 || f->n_layers < 1 || f->n_heads < 1 || f->hidden < 1 || f->capacity < 1 || f->topk < 1 ||
      f->max_tokens < 1 || f->ctrl_hidden < 1 || f->rebuild_max < 0 || f->rebuild_max >= f->capacity || (f->flags & ~uint32_t(ADORE_FLAG_NO_RECURRENCE | ADORE_FLAG_SCORE_FROM_ATTENTION | ADORE_FLAG_RELATIVE_POSITION)) != 0 ||
      ((f->flags & ADORE_FLAG_SCORE_FROM_ATTENTION) && (f->flags & ADORE_FLAG_RELATIVE_POSITION)) ||
      !(f->pos_scale > 0.f) || f->rope_theta < 0.f)
    return ADORE_ERR_INVALID_ARG;
  if (f->dtype != ADORE_F32 && f->dtype != ADORE_BF16) return ADORE_ERR_INVALID_ARG;
  if (f->rebuild_mode != ADORE_REBUILD_POLICY && f->rebuild_mode != ADORE_REBUILD_EXPLICIT) return ADORE_ERR_INVALID_ARG;
  if (f->head_dim != 64 && f->head_dim != 128) return ADORE_ERR_UNSUPPORTED;
  if (f->capacity > 4096 || f->max_tokens > 8192 || f->ctrl_hidden > 256 || f->hidden % 64 != 0)
    return ADORE_ERR_UNSUPPORTED;
  return ADORE_OK;
}

}  // namespace

namespace {

// Launches, on the controller stream, the copy of the new token's row into the token store and the controller of
// token n (gates, then GRU + MLP + score), and on `sel` the step's selection and row table. Both streams must already
// wait for the point of the main stream the step starts from; with `ctrl_after_attention` the controller also waits
// for ev_attn, which the caller has recorded. Records ev_xrow (x_new has been read) and, if `sel` is a side stream,
// ev_join (map, lists and row table are written); the main stream has to wait for both.
adore_status_t launch_controller_and_selection(adore_cache* c, const void* x_new, const int32_t* explicit_list,
                                             const int32_t* explicit_count, int32_t r_in, cudaStream_t sel,
                                             bool early_gather, bool ctrl_after_attention) {
  const adore_config_t& f = c->cfg;
  const bool ex = f.rebuild_mode == ADORE_REBUILD_EXPLICIT;
  adore_status_t st;
  StageScope scope(c, 1);
  const bool controller = !(f.flags & ADORE_FLAG_SCORE_FROM_ATTENTION);   // else the scores come from the attention
  {
    const int row_pieces = int(size_t(f.hidden) * c->esz / 16);
    store_row_kernel<<<f.batch, 256, 0, c->ctl>>>(static_cast<const uint4*>(x_new), static_cast<uint4*>(c->x_store), row_pieces,
                                                 static_cast<long long>(f.max_tokens) * row_pieces,
                                                 static_cast<long long>(c->n) * row_pieces);
    ++c->launches;
    CUDA_OK(cudaGetLastError());
    CUDA_OK(cudaEventRecord(c->ev_xrow, c->ctl));
    c->xrow_pending = true;
    if (ctrl_after_attention) CUDA_OK(cudaStreamWaitEvent(c->ctl, c->ev_attn, 0));
  }
  if (c->ctrl_pending) CUDA_OK(cudaStreamWaitEvent(sel, c->ev_ctrl, 0));   // scores of token n-1
  // The selection chain is what the step waits for, so it is queued first; the controller's launches follow.
  st = launch_rescore(c, c->n, sel);            // relative positions: the ranking below is the one seen from token n
  if (st != ADORE_OK) return st;
  const int P = ex ? pow2_at_least(r_in) : pow2_at_least(c->n);
  SelectParams sp = select_params(c, c->n, P, c->cur, 1 - c->cur);
  sp.explicit_list = ex && r_in > 0 ? explicit_list : nullptr;
  sp.explicit_count = ex && r_in > 0 ? explicit_count : nullptr;
  sp.r_in = r_in;
  // Short lists (the paper's R = 8): the last CTA of the launch also writes the rebuild's row table. Long lists keep the
  // table's own launch, one CTA per sequence: one CTA copying 16k entries took longer (16 us) than that launch (5 us).
  const bool table_in_select = f.rebuild_max > 0 && size_t(f.batch) * f.rebuild_max <= 4096;
  if (table_in_select) {
    sp.row_b = c->row_b; sp.row_tok = c->row_tok; sp.row_slot = c->row_slot; sp.row_total = c->row_total;
    sp.rows_accum = c->rows_accum; sp.done_count = c->sel_done;
  }
  const size_t smem = select_smem_bytes(f.capacity, P);
  select_kernel<<<f.batch, step_select_threads(c, P), smem, sel>>>(sp);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  if (!table_in_select) {
    st = launch_row_table(c, true, sel);
    if (st != ADORE_OK) return st;
  }
  c->joined = sel == c->stream;
  CUDA_OK(cudaEventRecord(c->ev_join, sel));     // the gather below is not part of what the main stream waits for
  // The gate product starts when the selection is done: side by side the two were measured several times slower
  // (gate product 14 -> 70 us, selection 18 -> 28 us at batch 16), whereas beside the rebuild GEMM it loses little.
  // (Also with per-stage timing on, where the selection runs on the main stream.)
  CUDA_OK(cudaStreamWaitEvent(c->ctl, c->ev_join, 0));
  // A short list's rows are copied out of the token store into the GEMM's compact input right away, beside the
  // attention, so that the rebuild that follows starts with its GEMM. Long lists are copied after the attention:
  // side by side the two slow each other down by more than the copy takes (measured at 15k rows: attention
  // 104 -> 193 us beside a copy that takes 35 us alone). (Not with per-stage timing on: there the copy stays
  // with the rebuild stage.)
  c->rows_gathered = false;
  {
    const int m_max = f.batch * f.rebuild_max;
    if (early_gather && !c->timing && f.dtype == ADORE_BF16 && tc_usable<__nv_bfloat16>(c->tc) && m_max > 0 && m_max <= 2048 &&
        size_t(m_max) <= c->tc.a_rows) {
      RebuildParams<__nv_bfloat16> gp{};
      gp.x_table = static_cast<const __nv_bfloat16*>(c->x_store); gp.seq_stride = f.max_tokens; gp.d = f.hidden;
      gp.row_b = c->row_b; gp.row_tok = c->row_tok; gp.row_total = c->row_total;
      CUDA_OK(launch_gather_tc<__nv_bfloat16>(c->tc, gp, m_max, sel));
      ++c->launches;
      c->rows_gathered = true;
      if (sel != c->stream) { CUDA_OK(cudaEventRecord(c->ev_gather, sel)); c->gather_pending = true; }   // the rebuild waits for it
    }
  }
  // the recurrent product rides in the gate product when the state has whole 32-element chunks and is not ignored
  const int hh_slices = (f.ctrl_hidden % kGateKInner == 0 && !(f.flags & ADORE_FLAG_NO_RECURRENCE))
                            ? (f.ctrl_hidden + kGateHhSlice - 1) / kGateHhSlice : 0;
  if (!controller) return ADORE_OK;
  {
    const size_t row0 = size_t(c->n) * f.hidden;        // token n of sequence 0 in the store [B][max_tokens][d]
    if (f.dtype == ADORE_F32)
      st = launch_gates<float>(c, static_cast<const float*>(c->x_store) + row0, f.max_tokens, 1, c->ksplit, c->ctl, hh_slices);
    else
      st = launch_gates<__nv_bfloat16>(c, static_cast<const __nv_bfloat16*>(c->x_store) + row0, f.max_tokens, 1, c->ksplit, c->ctl, hh_slices);
    if (st != ADORE_OK) return st;
  }
  RecurParams rp = recur_params(c, f.batch, 1, c->ksplit, c->n);
  rp.hh_slices = hh_slices;
  if (f.ctrl_hidden % 4 == 0) {
    // (an ordinary launch: while a programmatic dependent of the gate product was pending, kernels of the other streams
    // -- the new token's row, the gather -- were not started either)
    ctrl_decode_tail_kernel<<<f.batch, kTailThreads, ctrl_tail_smem_bytes(f.ctrl_hidden), c->ctl>>>(rp);
    CUDA_OK(cudaGetLastError());
  } else {                                            // rows that are not whole 16-byte pieces: the scalar-load kernel of the prompt scan
    ctrl_recur_kernel<<<f.batch, select_threads(c), ctrl_smem(c), c->ctl>>>(rp, 0, c->err);
    CUDA_OK(cudaGetLastError());
  }
  ++c->launches;
  CUDA_OK(cudaEventRecord(c->ev_ctrl, c->ctl));
  c->ctrl_pending = true;
  if (c->timing) { CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_ctrl, 0)); c->ctrl_pending = false; }
  return ADORE_OK;
}

}  // namespace

extern "C" {

const char* adore_status_string(adore_status_t s) {
  switch (s) {
    case ADORE_OK: return "ok";
    case ADORE_ERR_INVALID_ARG: return "invalid argument";
    case ADORE_ERR_OOM: return "out of memory";
    case ADORE_ERR_TOKEN_TABLE_FULL: return "token table full";
    case ADORE_ERR_STATE: return "call out of order";
    case ADORE_ERR_CUDA: return "CUDA call failed";
    case ADORE_ERR_DEVICE_FLAG: return "device error word set";
    case ADORE_ERR_TIMEOUT: return "bounded device wait gave up";
    case ADORE_ERR_UNSUPPORTED: return "unsupported shape";
  }
  return "unknown status";
}

adore_status_t adore_cache_create(const adore_config_t* cfg, const adore_controller_weights_t* w, void* cuda_stream,
                                  adore_cache_t** out) {
  if (!cfg || !w || !out) return ADORE_ERR_INVALID_ARG;
  *out = nullptr;
  adore_status_t st = check_config(cfg);
  if (st != ADORE_OK) return st;
  if (!w->gru_w_ih || !w->gru_w_hh || !w->gru_b_ih || !w->gru_b_hh || !w->pos_w || !w->pos_b || !w->mlp_w1 ||
      !w->mlp_b1 || !w->mlp_w2 || !w->mlp_b2)
    return ADORE_ERR_INVALID_ARG;
  adore_cache* c = new (std::nothrow) adore_cache();
  if (!c) return ADORE_ERR_OOM;
  c->cfg = *cfg;
  c->stream = static_cast<cudaStream_t>(cuda_stream);
  c->esz = cfg->dtype == ADORE_F32 ? 4 : 2;
  c->w_kv.assign(cfg->n_layers, nullptr);
  const adore_config_t& f = c->cfg;
  const size_t B = f.batch, C = f.capacity, MT = f.max_tokens, h = f.ctrl_hidden, d = f.hidden, G = 3 * h;
  const size_t kv_bytes = size_t(f.n_layers) * B * f.n_heads * C * f.head_dim * c->esz;
  const size_t rmax1 = f.rebuild_max > 0 ? f.rebuild_max : 1;
#define TRY(x) do { st = (x); if (st != ADORE_OK) { adore_cache_destroy(c); return st; } } while (0)
  TRY(dev_alloc(c, &c->Kc, kv_bytes, true));
  TRY(dev_alloc(c, &c->Vc, kv_bytes, true));
  TRY(dev_alloc(c, &c->x_store, B * MT * d * c->esz, false));
  TRY(dev_alloc(c, &c->z, B * h * sizeof(double), true));
  TRY(dev_alloc(c, &c->score, B * MT * sizeof(float), true));
  TRY(dev_alloc(c, &c->sigma, B * MT * sizeof(float), true));
  TRY(dev_alloc(c, &c->tok_slot, B * MT * sizeof(int), false));
  for (int i = 0; i < 2; ++i) {
    TRY(dev_alloc(c, &c->slot_tok[i], B * C * sizeof(int), false));
    TRY(dev_alloc(c, &c->slot_role[i], B * C, true));
    TRY(fill_i32(c, c->slot_tok[i], -1, B * C));
  }
  TRY(fill_i32(c, c->tok_slot, -1, B * MT));
  TRY(dev_alloc(c, &c->admit_slot, B * sizeof(int), true));
  TRY(dev_alloc(c, &c->evicted_tok, B * sizeof(int), true));
  TRY(dev_alloc(c, &c->rebuild_tok, B * rmax1 * sizeof(int), true));
  TRY(dev_alloc(c, &c->rebuild_slot, B * rmax1 * sizeof(int), true));
  TRY(dev_alloc(c, &c->rebuild_count, B * sizeof(int), true));
  TRY(dev_alloc(c, &c->row_b, B * rmax1 * sizeof(int), true));
  TRY(dev_alloc(c, &c->row_tok, B * rmax1 * sizeof(int), true));
  TRY(dev_alloc(c, &c->row_slot, B * rmax1 * sizeof(int), true));
  TRY(dev_alloc(c, &c->row_total, sizeof(int), true));
  TRY(dev_alloc(c, &c->frow_b, B * C * sizeof(int), true));
  TRY(dev_alloc(c, &c->frow_tok, B * C * sizeof(int), true));
  TRY(dev_alloc(c, &c->frow_slot, B * C * sizeof(int), true));
  TRY(dev_alloc(c, &c->frow_total, sizeof(int), true));
  TRY(dev_alloc(c, &c->rows_accum, sizeof(unsigned long long), true));
  TRY(dev_alloc(c, &c->sel_done, sizeof(unsigned), true));
  {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&c->sms, cudaDevAttrMultiProcessorCount, dev);
  }
  TRY(dev_alloc(c, &c->err, sizeof(unsigned), true));
  if (f.flags & ADORE_FLAG_SCORE_FROM_ATTENTION)
    TRY(dev_alloc(c, &c->w_internal, B * f.n_heads * (C + 1) * sizeof(float), true));
  // decode splits the d-long dot products into k-slices (whole 32-element chunks) so that the launch has about one CTA per SM
  {
    const bool wide = int(B) >= kGateWideMinRows;
    const int tiles = wide ? int((G + kGateWideG - 1) / kGateWideG) * int((B + kGateWideR - 1) / kGateWideR)
                           : int((G + kGateTileG - 1) / kGateTileG) * int((B + kGateTileR - 1) / kGateTileR);
    const int chunks = int(d) / kGateKInner;
    const int ks_cap = h % 4 == 0 ? 64 : 32;       // odd widths go through the prompt kernel, which adds at most 32 slices
    const int ks_max = std::max(1, std::min(ks_cap, c->sms / std::max(1, tiles)));
    const int slice_chunks = (chunks + ks_max - 1) / ks_max;
    const int ks = (chunks + slice_chunks - 1) / slice_chunks;
    c->ksplit = ks;
    const size_t rows_prefill = std::min<size_t>(B * MT, std::max<size_t>(kMaxPrefillRows, B));
    c->part_doubles = std::max<size_t>(size_t(ks + 4) * B, rows_prefill) * G;   // + 4: the recurrent product's slices (d' <= 256)
    TRY(dev_alloc(c, &c->part, c->part_doubles * sizeof(double), false));
  }
  TRY(upload(c, &c->w_hh, w->gru_w_hh, G * h));
  TRY(upload(c, &c->w1, w->mlp_w1, h * h));
  TRY(upload(c, &c->w_ih, w->gru_w_ih, G * d));
  TRY(upload(c, &c->b_ih, w->gru_b_ih, G));
  TRY(upload(c, &c->b_hh, w->gru_b_hh, G));
  TRY(upload(c, &c->pos_w, w->pos_w, h));
  TRY(upload(c, &c->pos_b, w->pos_b, h));
  TRY(upload(c, &c->b1, w->mlp_b1, h));
  TRY(upload(c, &c->w2, w->mlp_w2, h));
  TRY(upload(c, &c->b2, w->mlp_b2, 1));
  if (f.flags & ADORE_FLAG_RELATIVE_POSITION) {
    TRY(dev_alloc(c, &c->a_tab, B * MT * h * sizeof(double), true));
    TRY(dev_alloc(c, &c->c_vec, h * sizeof(double), false));
    ctrl_position_direction_kernel<<<int((h + 127) / 128), 128, 0, c->stream>>>(c->w1, c->pos_w, c->c_vec, int(h));
    ++c->launches;
    if (cudaGetLastError() != cudaSuccess) { adore_cache_destroy(c); return ADORE_ERR_CUDA; }
  }
  if (f.rope_theta != 0.f) {   // rotation angle of pair j at position p: p * theta^(-2j/dh)
    const size_t half = f.head_dim / 2;
    std::vector<float> cs(MT * half), sn(MT * half);
    for (size_t j = 0; j < half; ++j) {
      const double inv = std::pow(double(f.rope_theta), -2.0 * double(j) / double(f.head_dim));
      for (size_t pos = 0; pos < MT; ++pos) {
        cs[pos * half + j] = float(std::cos(double(pos) * inv));
        sn[pos * half + j] = float(std::sin(double(pos) * inv));
      }
    }
    TRY(upload(c, &c->rope_cos, cs.data(), MT * half));
    TRY(upload(c, &c->rope_sin, sn.data(), MT * half));
  }
  // opt in to large dynamic shared memory where a kernel may need it
  {
    const int big = 227 * 1024;
    cudaFuncSetAttribute(ctrl_recur_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    cudaFuncSetAttribute(ctrl_gates_wide_kernel<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGateWideSmem));
    cudaFuncSetAttribute(ctrl_gates_wide_kernel<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kGateWideSmem));
    cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    cudaFuncSetAttribute(bulk_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, big);
    if (cudaGetLastError() != cudaSuccess) { adore_cache_destroy(c); return ADORE_ERR_CUDA; }
  }
  // the side streams carry short kernels that the step's critical path waits for: their CTAs go ahead of the
  // attention kernel's pending ones
  int prio_low = 0, prio_high = 0;
  cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high);
  if (cudaStreamCreateWithPriority(&c->aux, cudaStreamNonBlocking, prio_high) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithPriority(&c->ctl, cudaStreamNonBlocking, prio_high) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_xrow, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_gather, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_attn, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_ctrl, cudaEventDisableTiming) != cudaSuccess ||
      cudaStreamCreateWithFlags(&c->copy, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_copy, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&c->ev_out, cudaEventDisableTiming) != cudaSuccess) {
    adore_cache_destroy(c);
    return ADORE_ERR_CUDA;
  }
  if (f.n_layers > 1) {
    bool ok = cudaStreamCreateWithFlags(&c->rb, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_rb_fork, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&c->ev_step_open, cudaEventDisableTiming) == cudaSuccess;
    c->rb_pending.assign(size_t(f.n_layers), char(0));
    for (int l = 0; ok && l < f.n_layers; ++l) {
      cudaEvent_t e = nullptr;
      ok = cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
      if (ok) c->ev_rebuilt.push_back(e);
    }
    if (!ok) { adore_cache_destroy(c); return ADORE_ERR_CUDA; }
  }
  if (f.dtype == ADORE_BF16) {
    st = tc_init(c->tc, f, c->owned, c->stream);
    if (st != ADORE_OK) { adore_cache_destroy(c); return st; }
    if (c->tc.encode != nullptr && (f.head_dim == 64 || f.head_dim == 128)) {
      // tensor maps over each layer's key and value cache for the kernel with several query rows per pair
      const size_t layer_elems = B * f.n_heads * C * f.head_dim;
      c->map_k.resize(f.n_layers);
      c->map_v.resize(f.n_layers);
      bool ok = true;
      for (int l = 0; l < f.n_layers && ok; ++l) {
        const cuuint64_t dims[2] = {cuuint64_t(f.head_dim), cuuint64_t(B * f.n_heads * C)};
        const cuuint64_t strides[1] = {cuuint64_t(f.head_dim) * 2};
        const cuuint32_t box[2] = {64u, uint32_t(kRowsTile)};
        const cuuint32_t estr[2] = {1, 1};
        void* bases[2] = {static_cast<__nv_bfloat16*>(c->Kc) + l * layer_elems, static_cast<__nv_bfloat16*>(c->Vc) + l * layer_elems};
        CUtensorMap* maps[2] = {&c->map_k[l], &c->map_v[l]};
        for (int j = 0; j < 2; ++j)
          ok = ok && c->tc.encode(maps[j], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bases[j], dims, strides, box, estr,
                                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
      }
      if (!ok) { c->map_k.clear(); c->map_v.clear(); }
    }
  }
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) { adore_cache_destroy(c); return ADORE_ERR_CUDA; }
#undef TRY
  *out = c;
  return ADORE_OK;
}

adore_status_t adore_cache_destroy(adore_cache_t* c) {
  if (!c) return ADORE_OK;
  cudaStreamSynchronize(c->stream);
  if (c->aux) { cudaStreamSynchronize(c->aux); cudaStreamDestroy(c->aux); }
  if (c->ctl) { cudaStreamSynchronize(c->ctl); cudaStreamDestroy(c->ctl); }
  if (c->rb) { cudaStreamSynchronize(c->rb); cudaStreamDestroy(c->rb); }
  if (c->d2h) { cudaStreamSynchronize(c->d2h); cudaStreamDestroy(c->d2h); }
  if (c->ev_rb_fork) cudaEventDestroy(c->ev_rb_fork);
  if (c->ev_step_open) cudaEventDestroy(c->ev_step_open);
  for (cudaEvent_t e : c->ev_rebuilt) cudaEventDestroy(e);
  if (c->ev_xrow) cudaEventDestroy(c->ev_xrow);
  if (c->ev_gather) cudaEventDestroy(c->ev_gather);
  if (c->ev_attn) cudaEventDestroy(c->ev_attn);
  if (c->ev_ctrl) cudaEventDestroy(c->ev_ctrl);
  if (c->copy) { cudaStreamSynchronize(c->copy); cudaStreamDestroy(c->copy); }
  if (c->ev_copy) cudaEventDestroy(c->ev_copy);
  if (c->ev_out) cudaEventDestroy(c->ev_out);
  if (c->ev_fork) cudaEventDestroy(c->ev_fork);
  if (c->ev_join) cudaEventDestroy(c->ev_join);
  for (void* p : c->owned) cudaFree(p);
  for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : c->grp_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_stage_free) cudaEventDestroy(e);
  cudaGetLastError();
  delete c;
  return ADORE_OK;
}

adore_status_t adore_cache_set_projection(adore_cache_t* c, int32_t layer, const void* w_kv) {
  if (!c || !w_kv || layer < 0 || layer >= c->cfg.n_layers) return ADORE_ERR_INVALID_ARG;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;   // a rebuild beside the main stream may still read the old weights
  if (reinterpret_cast<uintptr_t>(w_kv) % 16 != 0) return ADORE_ERR_INVALID_ARG;
  c->w_kv[layer] = w_kv;
  if (c->cfg.dtype == ADORE_BF16) return tc_set_weights(c->tc, layer, w_kv);
  return ADORE_OK;
}

adore_status_t adore_cache_append_tokens(adore_cache_t* c, const void* x, int32_t T) {
  if (!c || !x || T < 1) return ADORE_ERR_INVALID_ARG;
  if (c->n != 0) return ADORE_ERR_STATE;
  const adore_config_t& f = c->cfg;
  if (T > f.max_tokens) return ADORE_ERR_TOKEN_TABLE_FULL;
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  const size_t row = size_t(f.hidden) * c->esz;
  CUDA_OK(cudaMemcpy2DAsync(c->x_store, size_t(f.max_tokens) * row, x, size_t(T) * row, size_t(T) * row, f.batch,
                            cudaMemcpyDeviceToDevice, c->stream));
  int chunk = int(c->part_doubles / (size_t(3) * f.ctrl_hidden) / f.batch);
  if (chunk < 1) chunk = 1;
  // with the attention as the score source a prompt token has earned nothing yet: all scores stay zero
  for (int t0 = 0; t0 < T && !(f.flags & ADORE_FLAG_SCORE_FROM_ATTENTION); t0 += chunk) {
    const int tc = std::min(chunk, T - t0);
    adore_status_t st;
    if (f.dtype == ADORE_F32)
      st = launch_gates<float>(c, static_cast<const float*>(c->x_store) + size_t(t0) * f.hidden, f.max_tokens, tc, 1, c->stream);
    else
      st = launch_gates<__nv_bfloat16>(c, static_cast<const __nv_bfloat16*>(c->x_store) + size_t(t0) * f.hidden,
                                       f.max_tokens, tc, 1, c->stream);
    if (st != ADORE_OK) return st;
    RecurParams rp = recur_params(c, f.batch * tc, tc, 1, t0);
    ctrl_recur_kernel<<<f.batch, select_threads(c), ctrl_smem(c), c->stream>>>(rp, ctrl_resident_ok(f.ctrl_hidden) ? 1 : 0, c->err);
    ++c->launches;
    CUDA_OK(cudaGetLastError());
  }
  {                                             // relative positions: the prompt as seen from its last token
    adore_status_t st = launch_rescore(c, T - 1, c->stream);
    if (st != ADORE_OK) return st;
  }
  const int P = pow2_at_least(T);
  SelectParams sp = select_params(c, T, P, c->cur, c->cur);
  bulk_select_kernel<<<f.batch, select_threads(c), select_smem_bytes(f.capacity, P), c->stream>>>(sp);
  ++c->launches;
  CUDA_OK(cudaGetLastError());
  {
    adore_status_t st = launch_row_table(c, false, c->stream);
    if (st != ADORE_OK) return st;
  }
  c->n = T;
  c->attn = c->cur;
  for (int l = 0; l < f.n_layers; ++l)
    if (c->w_kv[l]) {
      adore_status_t st = fill_layer_impl(c, l, nullptr);
      if (st != ADORE_OK) return st;
    }
  return ADORE_OK;
}

adore_status_t adore_cache_fill_layer(adore_cache_t* c, int32_t layer, const void* x_table) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || misaligned16(x_table)) return ADORE_ERR_INVALID_ARG;
  if (!c->w_kv[layer]) return ADORE_ERR_STATE;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  return fill_layer_impl(c, layer, x_table);
}

adore_status_t adore_decode_step(adore_cache_t* c, int32_t layer, const void* q, const void* k_new, const void* v_new,
                                 const void* x_new, const int32_t* explicit_list, const int32_t* explicit_count,
                                 int32_t r_in, void* out, float* weights) {
  if (!c || !q || !k_new || !v_new || !out || layer < 0 || layer >= c->cfg.n_layers) return ADORE_ERR_INVALID_ARG;
  if (misaligned16(q) || misaligned16(k_new) || misaligned16(v_new) || misaligned16(out) || (layer == 0 && misaligned16(x_new)))
    return ADORE_ERR_INVALID_ARG;
  const adore_config_t& f = c->cfg;
  const bool from_attention = (f.flags & ADORE_FLAG_SCORE_FROM_ATTENTION) != 0;
  if (from_attention && !weights) weights = c->w_internal;
  if (layer == 0) {
    if (!x_new) return ADORE_ERR_INVALID_ARG;
    if (c->n >= f.max_tokens) return ADORE_ERR_TOKEN_TABLE_FULL;
    const bool ex = f.rebuild_mode == ADORE_REBUILD_EXPLICIT;
    if (r_in < 0 || (ex && r_in > 0 && (!explicit_list || !explicit_count))) return ADORE_ERR_INVALID_ARG;
    if (ex && r_in > 8192) return ADORE_ERR_UNSUPPORTED;
    // Three things start here and run side by side: the attention of this layer on the main stream, reading the
    // cache through the previous slot map; the selection on one side stream (it needs the scores of tokens < n
    // only); the controller of token n on another (gate products, then GRU + MLP + score). The new token's row is
    // written once attention and selection are done. The controller may run on past this step: the next step's
    // selection waits for it, and so does every call that reads or replaces the controller state.
    // (With per-stage timing on, the selection stays on the main stream and the controller is joined before the
    // stage's closing event, so that the stage times add up.)
    cudaStream_t sel = c->timing ? c->stream : c->aux;
    adore_status_t st;
    // Rebuilds of the previous step may still run beside the main stream: the attention below needs layer 0's, the
    // selection chain (which rewrites the row table and the gather buffer they read) needs all of them.
    if (c->timing) { if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA; }
    else if (wait_rebuild(c, 0, c->stream) != ADORE_OK) return ADORE_ERR_CUDA;
    if (!c->timing && c->rb_last >= 0) {
      CUDA_OK(cudaStreamWaitEvent(sel, c->ev_rebuilt[c->rb_last], 0));
      // the selection joins the main stream before this step's first rebuild: from then on the main stream is
      // behind every earlier rebuild too
      c->rb_last = -1;
      std::fill(c->rb_pending.begin(), c->rb_pending.end(), char(0));
    }
    // the attention is the longest of the three and is launched first; the side streams start from the same point
    // (with per-stage timing on: from the end of the attention, so that no stage overlaps another)
    if (!c->timing) CUDA_OK(cudaEventRecord(c->ev_fork, c->stream));
    if (group_mark(c, 0, c->stream) != ADORE_OK) return ADORE_ERR_CUDA;
    c->attn = c->cur;
    st = f.dtype == ADORE_F32 ? launch_attention<float>(c, 0, q, k_new, v_new, out, weights, false)
                              : launch_attention<__nv_bfloat16>(c, 0, q, k_new, v_new, out, weights, false);
    if (st != ADORE_OK) return st;
    if (c->timing) CUDA_OK(cudaEventRecord(c->ev_fork, c->stream));
    if (sel != c->stream) CUDA_OK(cudaStreamWaitEvent(sel, c->ev_fork, 0));
    // The controller's float64 products would take SM time from the attention, which fills the GPU and is on the step's
    // critical path, while their result is first needed by the NEXT step's selection: they start when the attention
    // of layer 0 is done and run beside what follows it (the gather of a long rebuild list, the next layers).
    // The copy of the new token's row into the store, which is all that reads x_new, does start at the fork.
    CUDA_OK(cudaEventRecord(c->ev_attn, c->stream));
    CUDA_OK(cudaStreamWaitEvent(c->ctl, c->ev_fork, 0));
    st = launch_controller_and_selection(c, x_new, explicit_list, explicit_count, r_in, sel, true, true);
    if (st != ADORE_OK) return st;
    if (group_mark(c, 2, c->ctl) != ADORE_OK) return ADORE_ERR_CUDA;
    c->cur = 1 - c->cur;
    c->n += 1;
    c->step_layer0_done = 1;
  } else if (c->step_layer0_done != 1) {
    return ADORE_ERR_STATE;       // no step open, or one opened by adore_step_begin
  }
  if (layer != 0) {
    if (wait_rebuild(c, layer, c->stream) != ADORE_OK) return ADORE_ERR_CUDA;
    adore_status_t st = f.dtype == ADORE_F32 ? launch_attention<float>(c, layer, q, k_new, v_new, out, weights, true)
                                             : launch_attention<__nv_bfloat16>(c, layer, q, k_new, v_new, out, weights, true);
    if (st == ADORE_OK && from_attention) st = launch_add_attention(c, weights);
    if (st == ADORE_OK && layer == f.n_layers - 1) st = group_mark(c, 1, c->stream);
    return st;
  }
  if (!c->joined) CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_join, 0));
  c->joined = true;
  if (c->xrow_pending) {          // x_new is the caller's again once the main stream has passed this point
    CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_xrow, 0));
    c->xrow_pending = false;
  }
  {
    StageScope scope(c, 3);
    const size_t row_bytes = size_t(f.head_dim) * c->esz;
    admit_rows_kernel<<<f.batch * f.n_heads, 32, 0, c->stream>>>(
        static_cast<unsigned char*>(c->Kc), static_cast<unsigned char*>(c->Vc), static_cast<const unsigned char*>(k_new),
        static_cast<const unsigned char*>(v_new), c->admit_slot, f.n_heads, f.capacity, int(row_bytes), c->err);
    ++c->launches;
    CUDA_OK(cudaGetLastError());
  }
  // after the join: this step's selection has read the scores it ranks by, the weights count from the next step on
  if (from_attention) {
    adore_status_t st = launch_add_attention(c, weights);
    if (st != ADORE_OK) return st;
  }
  if (f.n_layers == 1) return group_mark(c, 1, c->stream);
  return ADORE_OK;
}

adore_status_t adore_step_begin(adore_cache_t* c, const void* x_new, const int32_t* explicit_list,
                                const int32_t* explicit_count, int32_t r_in) {
  if (!c || !x_new || misaligned16(x_new)) return ADORE_ERR_INVALID_ARG;
  const adore_config_t& f = c->cfg;
  if (f.flags & ADORE_FLAG_SCORE_FROM_ATTENTION) return ADORE_ERR_UNSUPPORTED;   // defined for the attend-first step
  if (c->n >= f.max_tokens) return ADORE_ERR_TOKEN_TABLE_FULL;
  const bool ex = f.rebuild_mode == ADORE_REBUILD_EXPLICIT;
  if (r_in < 0 || (ex && r_in > 0 && (!explicit_list || !explicit_count))) return ADORE_ERR_INVALID_ARG;
  if (ex && r_in > 8192) return ADORE_ERR_UNSUPPORTED;
  // nothing of this step has run yet: selection and controller start side by side, the main stream waits for the
  // selection (the rebuild and the attention of the step read its map) and for the kernel that reads x_new
  cudaStream_t sel = c->timing ? c->stream : c->aux;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  CUDA_OK(cudaEventRecord(c->ev_fork, c->stream));
  if (sel != c->stream) CUDA_OK(cudaStreamWaitEvent(sel, c->ev_fork, 0));
  CUDA_OK(cudaStreamWaitEvent(c->ctl, c->ev_fork, 0));
  adore_status_t st = launch_controller_and_selection(c, x_new, explicit_list, explicit_count, r_in, sel, false, false);
  if (st != ADORE_OK) return st;
  if (!c->joined) CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_join, 0));
  c->joined = true;
  CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_xrow, 0));      // x_new has been read
  c->xrow_pending = false;
  if (c->ev_step_open) CUDA_OK(cudaEventRecord(c->ev_step_open, c->stream));
  c->cur = 1 - c->cur;
  c->attn = c->cur;             // this step's attention reads the NEW map
  c->n += 1;
  c->step_layer0_done = 2;      // a rebuild-first step is open
  return ADORE_OK;
}

adore_status_t adore_attend_rows(adore_cache_t* c, int32_t layer, const void* q_rows, const void* k_new, const void* v_new,
                                 void* out, float* weights) {
  if (!c || !q_rows || !k_new || !v_new || !out || layer < 0 || layer >= c->cfg.n_layers) return ADORE_ERR_INVALID_ARG;
  if (misaligned16(q_rows) || misaligned16(k_new) || misaligned16(v_new) || misaligned16(out)) return ADORE_ERR_INVALID_ARG;
  if (c->step_layer0_done != 2) return ADORE_ERR_STATE;
  if (wait_rebuild(c, layer, c->stream) != ADORE_OK) return ADORE_ERR_CUDA;   // this layer's rows may come from the side stream
  const adore_config_t& f = c->cfg;
  const int rows_q = f.rebuild_max + 1;
  return f.dtype == ADORE_F32 ? launch_attention<float>(c, layer, q_rows, k_new, v_new, out, weights, true, rows_q)
                              : launch_attention<__nv_bfloat16>(c, layer, q_rows, k_new, v_new, out, weights, true, rows_q);
}

namespace {

adore_status_t decode_step_host_impl(adore_cache_t* c, int32_t layer, const void* q, const void* k_new,
                                     const void* v_new, const void* x_new, const int32_t* explicit_list,
                                     const int32_t* explicit_count, int32_t r_in, void* out, float* weights,
                                     bool then_rebuild, const void* x_table) {
  if (!c || !q || !k_new || !v_new || !out) return ADORE_ERR_INVALID_ARG;
  const adore_config_t& f = c->cfg;
  const size_t qb = size_t(f.batch) * f.n_heads * f.head_dim * c->esz, xb = size_t(f.batch) * f.hidden * c->esz;
  if (!c->h_q) {
    adore_status_t sa = alloc_group(c, {{&c->h_q, qb}, {&c->h_k, qb}, {&c->h_v, qb}, {&c->h_out, qb}, {&c->h_x, xb},
                                        {reinterpret_cast<void**>(&c->h_list), size_t(f.batch) * f.max_tokens * sizeof(int)},
                                        {reinterpret_cast<void**>(&c->h_count), size_t(f.batch) * sizeof(int)}});
    if (sa != ADORE_OK) return sa;
  }
  if (r_in < 0 || r_in > f.max_tokens) return ADORE_ERR_INVALID_ARG;
  // The staging buffers are free (the previous call waited for every kernel that read them), so the
  // uploads need not queue behind the rebuild that may still be running on the main stream.
  CUDA_OK(cudaMemcpyAsync(c->h_q, q, qb, cudaMemcpyHostToDevice, c->copy));
  CUDA_OK(cudaMemcpyAsync(c->h_k, k_new, qb, cudaMemcpyHostToDevice, c->copy));
  CUDA_OK(cudaMemcpyAsync(c->h_v, v_new, qb, cudaMemcpyHostToDevice, c->copy));
  const bool lists = layer == 0 && explicit_list && explicit_count && r_in > 0;
  if (layer == 0) {
    if (!x_new) return ADORE_ERR_INVALID_ARG;
    CUDA_OK(cudaMemcpyAsync(c->h_x, x_new, xb, cudaMemcpyHostToDevice, c->copy));
    if (lists) {
      CUDA_OK(cudaMemcpyAsync(c->h_list, explicit_list, size_t(f.batch) * r_in * sizeof(int), cudaMemcpyHostToDevice, c->copy));
      CUDA_OK(cudaMemcpyAsync(c->h_count, explicit_count, size_t(f.batch) * sizeof(int), cudaMemcpyHostToDevice, c->copy));
    }
  }
  CUDA_OK(cudaEventRecord(c->ev_copy, c->copy));
  CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_copy, 0));
  adore_status_t st = adore_decode_step(c, layer, c->h_q, c->h_k, c->h_v, c->h_x, lists ? c->h_list : nullptr,
                                        lists ? c->h_count : nullptr, lists ? r_in : 0, c->h_out, weights);
  if (st != ADORE_OK) return st;
  CUDA_OK(cudaMemcpyAsync(out, c->h_out, qb, cudaMemcpyDeviceToHost, c->stream));
  if (!then_rebuild) {
    CUDA_OK(cudaStreamSynchronize(c->stream));
    return ADORE_OK;
  }
  // The rebuild is queued BEFORE the host waits, and the host waits for the copy of `out` only: the GPU goes from the
  // attention straight into the GEMM while the caller already works on `out` (and uploads the next step's inputs).
  // Every kernel that reads the staging buffers has finished by the time `out` has arrived.
  CUDA_OK(cudaEventRecord(c->ev_out, c->stream));
  st = adore_rebuild(c, layer, x_table);
  if (st != ADORE_OK) return st;
  CUDA_OK(cudaEventSynchronize(c->ev_out));
  return ADORE_OK;
}

}  // namespace

adore_status_t adore_decode_step_host(adore_cache_t* c, int32_t layer, const void* q, const void* k_new,
                                      const void* v_new, const void* x_new, const int32_t* explicit_list,
                                      const int32_t* explicit_count, int32_t r_in, void* out, float* weights) {
  return decode_step_host_impl(c, layer, q, k_new, v_new, x_new, explicit_list, explicit_count, r_in, out, weights, false, nullptr);
}

adore_status_t adore_decode_rebuild_host(adore_cache_t* c, int32_t layer, const void* q, const void* k_new,
                                         const void* v_new, const void* x_new, const int32_t* explicit_list,
                                         const int32_t* explicit_count, int32_t r_in, const void* x_table, void* out,
                                         float* weights) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !c->w_kv[layer]) return c ? ADORE_ERR_STATE : ADORE_ERR_INVALID_ARG;
  return decode_step_host_impl(c, layer, q, k_new, v_new, x_new, explicit_list, explicit_count, r_in, out, weights, true, x_table);
}

adore_status_t adore_decode_rebuild_host_queued(adore_cache_t* c, int32_t layer, const void* q, const void* k_new,
                                                const void* v_new, const void* x_new, const int32_t* explicit_list,
                                                const int32_t* explicit_count, int32_t r_in, const void* x_table, void* out,
                                                float* weights) {
  if (!c || !q || !k_new || !v_new || !out || layer < 0 || layer >= c->cfg.n_layers) return ADORE_ERR_INVALID_ARG;
  if (!c->w_kv[layer]) return ADORE_ERR_STATE;
  const adore_config_t& f = c->cfg;
  const size_t qb = size_t(f.batch) * f.n_heads * f.head_dim * c->esz, xb = size_t(f.batch) * f.hidden * c->esz;
  if (r_in < 0 || r_in > f.max_tokens) return ADORE_ERR_INVALID_ARG;
  if (layer == 0 && !x_new) return ADORE_ERR_INVALID_ARG;
  if (!c->hq_all) {
    // stream and events first (cheap to undo), the buffers last: the set exists as a whole or not at all
    cudaStream_t d2h = nullptr;
    std::vector<cudaEvent_t> evs;
    bool ok = cudaStreamCreateWithFlags(&d2h, cudaStreamNonBlocking) == cudaSuccess;
    for (int l = 0; ok && l < f.n_layers; ++l) {
      cudaEvent_t e = nullptr;
      ok = cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
      if (ok) { evs.push_back(e); ok = cudaEventRecord(e, c->stream) == cudaSuccess; }
    }
    adore_status_t sa = ok ? alloc_group(c, {{reinterpret_cast<void**>(&c->hq_all), size_t(f.n_layers) * 4 * qb}, {&c->hq_x, xb},
                                             {reinterpret_cast<void**>(&c->hq_list), size_t(f.batch) * f.max_tokens * sizeof(int)},
                                             {reinterpret_cast<void**>(&c->hq_count), size_t(f.batch) * sizeof(int)}})
                           : ADORE_ERR_CUDA;
    if (sa != ADORE_OK) {
      for (cudaEvent_t e : evs) cudaEventDestroy(e);
      if (d2h) cudaStreamDestroy(d2h);
      cudaGetLastError();
      return sa;
    }
    c->d2h = d2h;
    c->ev_stage_free = evs;
  }
  unsigned char* set = c->hq_all + size_t(layer) * 4 * qb;
  void *dq = set, *dk = set + qb, *dv = set + 2 * qb, *dout = set + 3 * qb;
  // the layer's staging set is free once the previous step's kernels that read it (and the copy of its `out`) are done
  CUDA_OK(cudaStreamWaitEvent(c->copy, c->ev_stage_free[layer], 0));
  CUDA_OK(cudaMemcpyAsync(dq, q, qb, cudaMemcpyHostToDevice, c->copy));
  CUDA_OK(cudaMemcpyAsync(dk, k_new, qb, cudaMemcpyHostToDevice, c->copy));
  CUDA_OK(cudaMemcpyAsync(dv, v_new, qb, cudaMemcpyHostToDevice, c->copy));
  const bool lists = layer == 0 && explicit_list && explicit_count && r_in > 0;
  if (layer == 0) {
    CUDA_OK(cudaMemcpyAsync(c->hq_x, x_new, xb, cudaMemcpyHostToDevice, c->copy));
    if (lists) {
      CUDA_OK(cudaMemcpyAsync(c->hq_list, explicit_list, size_t(f.batch) * r_in * sizeof(int), cudaMemcpyHostToDevice, c->copy));
      CUDA_OK(cudaMemcpyAsync(c->hq_count, explicit_count, size_t(f.batch) * sizeof(int), cudaMemcpyHostToDevice, c->copy));
    }
  }
  CUDA_OK(cudaEventRecord(c->ev_copy, c->copy));
  CUDA_OK(cudaStreamWaitEvent(c->stream, c->ev_copy, 0));
  adore_status_t st = adore_decode_step(c, layer, dq, dk, dv, c->hq_x, lists ? c->hq_list : nullptr,
                                        lists ? c->hq_count : nullptr, lists ? r_in : 0, dout, weights);
  if (st != ADORE_OK) return st;
  // by now the main stream is behind every kernel of this call that reads the staging set (the side streams were
  // joined inside adore_decode_step); `out` travels on its own stream, so that the next layer's attention follows
  // this one directly
  CUDA_OK(cudaEventRecord(c->ev_out, c->stream));
  CUDA_OK(cudaStreamWaitEvent(c->d2h, c->ev_out, 0));
  CUDA_OK(cudaMemcpyAsync(out, dout, qb, cudaMemcpyDeviceToHost, c->d2h));
  CUDA_OK(cudaEventRecord(c->ev_stage_free[layer], c->d2h));
  return adore_rebuild(c, layer, x_table);
}

adore_status_t adore_cache_wait_outputs(adore_cache_t* c) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (c->d2h && cudaStreamSynchronize(c->d2h) != cudaSuccess) return ADORE_ERR_CUDA;
  return ADORE_OK;
}

adore_status_t adore_rebuild(adore_cache_t* c, int32_t layer, const void* x_table) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || misaligned16(x_table)) return ADORE_ERR_INVALID_ARG;
  if (!c->w_kv[layer] || !c->step_layer0_done) return ADORE_ERR_STATE;
  const adore_config_t& f = c->cfg;
  // Attend-first order with several layers: this layer's rows are next read by the next step's attention of this
  // layer, so the rebuild goes to its own stream, behind everything queued so far (this layer's attention, the
  // selection, the new token's row), and the attention of the following layers runs beside it. (Not with per-stage
  // timing on, where stages must not overlap, and not in the rebuild-first order, whose attention reads these rows.)
  static const bool inline_only = dev_switch("ADORE_REBUILD_INLINE");
  // In the rebuild-first order the attention of layer l reads what rebuild(l) writes, but rebuild(l + 1) needs only the
  // step's selection: on the side stream it starts from the end of adore_step_begin and runs beside the attention of
  // layer l; adore_attend_rows(l + 1) waits for it.
  const bool beside = c->rb && !c->timing && !inline_only && c->step_layer0_done != 0 && f.batch * f.rebuild_max > 0;
  cudaStream_t stream = c->stream;
  if (beside) {
    if (c->step_layer0_done == 2) {
      CUDA_OK(cudaStreamWaitEvent(c->rb, c->ev_step_open, 0));
    } else {
      CUDA_OK(cudaEventRecord(c->ev_rb_fork, c->stream));
      CUDA_OK(cudaStreamWaitEvent(c->rb, c->ev_rb_fork, 0));
    }
    stream = c->rb;
  } else if (join_rebuilds(c) != ADORE_OK) {
    return ADORE_ERR_CUDA;
  }
  adore_status_t st =
      f.dtype == ADORE_F32
          ? launch_rebuild<float>(c, layer, x_table, c->row_b, c->row_tok, c->row_slot, c->row_total, f.batch * f.rebuild_max, true, stream)
          : launch_rebuild<__nv_bfloat16>(c, layer, x_table, c->row_b, c->row_tok, c->row_slot, c->row_total,
                                          f.batch * f.rebuild_max, true, stream);
  if (beside) {
    // recorded even after a failed launch: what did get queued on the side stream must be waited for all the same
    if (cudaEventRecord(c->ev_rebuilt[layer], c->rb) != cudaSuccess) return ADORE_ERR_CUDA;
    c->rb_pending[layer] = 1;
    c->rb_last = layer;
  }
  return st;
}

adore_status_t adore_cache_join(adore_cache_t* c) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  for (cudaEvent_t e : c->ev_stage_free) CUDA_OK(cudaStreamWaitEvent(c->stream, e, 0));   // queued `out` copies
  return ADORE_OK;
}

adore_status_t adore_cache_slot_map(adore_cache_t* c, const int32_t** slot_tok, const uint8_t** slot_role) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (slot_tok) *slot_tok = c->slot_tok[c->cur];
  if (slot_role) *slot_role = c->slot_role[c->cur];
  return ADORE_OK;
}

adore_status_t adore_cache_rebuild_list(adore_cache_t* c, const int32_t** tok, const int32_t** slot, const int32_t** count) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (tok) *tok = c->rebuild_tok;
  if (slot) *slot = c->rebuild_slot;
  if (count) *count = c->rebuild_count;
  return ADORE_OK;
}

adore_status_t adore_cache_step_info(adore_cache_t* c, const int32_t** admit_slot, const int32_t** evicted_tok) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (admit_slot) *admit_slot = c->admit_slot;
  if (evicted_tok) *evicted_tok = c->evicted_tok;
  return ADORE_OK;
}

adore_status_t adore_cache_scores(adore_cache_t* c, const float** score, const float** sigma) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (score) *score = c->score;
  if (sigma) *sigma = c->sigma;
  return ADORE_OK;
}

adore_status_t adore_cache_kv(adore_cache_t* c, int32_t layer, const void** k, const void** v) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return ADORE_ERR_INVALID_ARG;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;   // the rows may still be on their way on the side stream
  const size_t off = size_t(layer) * c->cfg.batch * c->cfg.n_heads * c->cfg.capacity * c->cfg.head_dim * c->esz;
  if (k) *k = static_cast<const unsigned char*>(c->Kc) + off;
  if (v) *v = static_cast<const unsigned char*>(c->Vc) + off;
  return ADORE_OK;
}

int32_t adore_cache_num_tokens(const adore_cache_t* c) { return c ? c->n : -1; }

int64_t adore_cache_launch_count(const adore_cache_t* c) { return c ? c->launches : -1; }

adore_status_t adore_cache_set_stage_timing(adore_cache_t* c, int32_t enable) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (enable < 0 || enable > 2) return ADORE_ERR_INVALID_ARG;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  c->timing = enable == 1;
  c->group_timing = enable == 2;
  return ADORE_OK;
}

adore_status_t adore_cache_group_times(adore_cache_t* c, double* ms, double* ms_main, int64_t* steps) {
  if (!c || !ms || !ms_main || !steps) return ADORE_ERR_INVALID_ARG;
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  for (size_t i = 0; i + 3 <= c->grp_used; i += 3) {
    float a = 0.f, b = 0.f;
    if (cudaEventElapsedTime(&a, c->grp_pool[i], c->grp_pool[i + 1]) != cudaSuccess) { cudaGetLastError(); continue; }   // a step left open
    if (cudaEventElapsedTime(&b, c->grp_pool[i], c->grp_pool[i + 2]) != cudaSuccess) { cudaGetLastError(); b = 0.f; }
    c->grp_ms += double(a > b ? a : b);
    c->grp_main_ms += double(a);
    c->grp_steps += 1;
  }
  c->grp_used = 0;
  *ms = c->grp_ms;
  *ms_main = c->grp_main_ms;
  *steps = c->grp_steps;
  c->grp_ms = c->grp_main_ms = 0;
  c->grp_steps = 0;
  return ADORE_OK;
}

adore_status_t adore_cache_stage_times(adore_cache_t* c, double* ms, int64_t* launches) {
  if (!c || !ms || !launches) return ADORE_ERR_INVALID_ARG;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  for (size_t i = 0; i < c->ev_stage.size(); ++i) {
    float t = 0.f;
    if (cudaEventElapsedTime(&t, c->ev_pool[2 * i], c->ev_pool[2 * i + 1]) != cudaSuccess) return ADORE_ERR_CUDA;
    c->stage_ms[c->ev_stage[i]] += double(t);
    c->stage_launches[c->ev_stage[i]] += 1;
  }
  c->ev_stage.clear();
  c->ev_used = 0;
  for (int s = 0; s < 4; ++s) {
    ms[s] = c->stage_ms[s];
    launches[s] = c->stage_launches[s];
    c->stage_ms[s] = 0;
    c->stage_launches[s] = 0;
  }
  return ADORE_OK;
}

adore_status_t adore_cache_rebuild_rows(adore_cache_t* c, int64_t* rows) {
  if (!c || !rows) return ADORE_ERR_INVALID_ARG;
  if (join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  unsigned long long v = 0;
  if (cudaMemcpy(&v, c->rows_accum, sizeof(v), cudaMemcpyDeviceToHost) != cudaSuccess) return ADORE_ERR_CUDA;
  *rows = int64_t(v);
  return ADORE_OK;
}

// ---- small-state snapshot ------------------------------------------------------------------------
namespace {

struct StateHeader {
  uint32_t magic, version;
  int32_t batch, capacity, rebuild_max, max_tokens, ctrl_hidden, n, cur, attn, step_open;
  uint32_t reserved[5];
};
static_assert(sizeof(StateHeader) == 64, "snapshot header is 64 bytes");
constexpr uint32_t kStateMagic = 0x54534441u;   // "ADST"

struct StateSection { void* ptr; size_t bytes; };

// Everything selection and scoring carry from step to step, in snapshot order (each section padded to 8 bytes).
std::vector<StateSection> state_sections(adore_cache* c) {
  const adore_config_t& f = c->cfg;
  const size_t B = f.batch, C = f.capacity, MT = f.max_tokens, h = f.ctrl_hidden;
  const size_t rmax1 = f.rebuild_max > 0 ? f.rebuild_max : 1;
  return {
      {c->slot_tok[0], B * C * sizeof(int)}, {c->slot_tok[1], B * C * sizeof(int)},
      {c->slot_role[0], B * C},              {c->slot_role[1], B * C},
      {c->tok_slot, B * MT * sizeof(int)},   {c->score, B * MT * sizeof(float)},  {c->sigma, B * MT * sizeof(float)},
      {c->z, B * h * sizeof(double)},
      {c->admit_slot, B * sizeof(int)},      {c->evicted_tok, B * sizeof(int)},
      {c->rebuild_tok, B * rmax1 * sizeof(int)}, {c->rebuild_slot, B * rmax1 * sizeof(int)}, {c->rebuild_count, B * sizeof(int)},
      {c->row_b, B * rmax1 * sizeof(int)},   {c->row_tok, B * rmax1 * sizeof(int)}, {c->row_slot, B * rmax1 * sizeof(int)},
      {c->row_total, sizeof(int)},
  };
}
// with relative positions the per-token Tanh inputs are state too (they are what later steps score from)
void add_relative_state(adore_cache* c, std::vector<StateSection>& sec) {
  if (c->a_tab) sec.push_back({c->a_tab, size_t(c->cfg.batch) * c->cfg.max_tokens * c->cfg.ctrl_hidden * sizeof(double)});
}
inline size_t pad8(size_t v) { return (v + 7) & ~size_t(7); }

// Index checks of a snapshot's integer sections before any of it reaches the device: the selection, the gather and the
// GEMM's scatter use these values as indices. `sec` is the cache's own section list (sizes only are used).
bool snapshot_consistent(const adore_config_t& f, const StateHeader& hd, const unsigned char* buf, const std::vector<StateSection>& sec) {
  std::vector<const unsigned char*> at(sec.size());
  size_t off = sizeof(StateHeader);
  for (size_t i = 0; i < sec.size(); ++i) { at[i] = buf + off; off += pad8(sec[i].bytes); }
  const int B = f.batch, C = f.capacity, MT = f.max_tokens, R = f.rebuild_max, m = C - R, n = hd.n;
  auto i32 = [&](size_t section, size_t idx) { int v; std::memcpy(&v, at[section] + idx * sizeof(int), sizeof(int)); return v; };
  for (int map = 0; map < 2; ++map)
    for (int b = 0; b < B; ++b) {
      int retained = 0, rebuilt = 0;
      for (int s = 0; s < C; ++s) {
        const int tok = i32(size_t(map), size_t(b) * C + s);
        const unsigned role = at[2 + map][size_t(b) * C + s];
        if (tok < -1 || tok >= n || role > ROLE_REBUILT || ((tok < 0) != (role == ROLE_EMPTY))) return false;
        retained += role == ROLE_RETAINED;
        rebuilt += role == ROLE_REBUILT;
      }
      if (retained > m || rebuilt > R) return false;
    }
  for (int b = 0; b < B; ++b) {
    for (int t = 0; t < MT; ++t) {
      const int s = i32(4, size_t(b) * MT + t);
      if (s < -1 || s >= C) return false;
    }
    const int adm = i32(8, b), ev = i32(9, b), cnt = i32(12, b);
    if (adm < -1 || adm >= C || ev < -1 || ev >= std::max(n, 1) || cnt < 0 || cnt > R) return false;
    for (int i = 0; i < cnt; ++i) {
      const int tok = i32(10, size_t(b) * R + i), slot = i32(11, size_t(b) * R + i);
      if (tok < 0 || tok >= n || slot < 0 || slot >= C) return false;
    }
  }
  const int total = i32(16, 0);
  if (total < 0 || total > B * R) return false;
  for (int i = 0; i < total; ++i) {
    const int b = i32(13, i), tok = i32(14, i), slot = i32(15, i);
    if (b < 0 || b >= B || tok < 0 || tok >= n || slot < 0 || slot >= C) return false;
  }
  return true;
}

}  // namespace

adore_status_t adore_cache_export_state(adore_cache_t* c, void* host_buf, size_t* bytes) {
  if (!c || !bytes) return ADORE_ERR_INVALID_ARG;
  std::vector<StateSection> sec = state_sections(c);
  add_relative_state(c, sec);
  size_t need = sizeof(StateHeader);
  for (const StateSection& s : sec) need += pad8(s.bytes);
  if (!host_buf) { *bytes = need; return ADORE_OK; }
  if (*bytes < need) { *bytes = need; return ADORE_ERR_INVALID_ARG; }
  *bytes = need;
  // the side stream's work is joined into the main stream by the calls that use it; wait for both anyway
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  if (c->aux && cudaStreamSynchronize(c->aux) != cudaSuccess) return ADORE_ERR_CUDA;
  if (c->ctl && cudaStreamSynchronize(c->ctl) != cudaSuccess) return ADORE_ERR_CUDA;
  StateHeader hd{};
  hd.magic = kStateMagic; hd.version = 1;
  hd.batch = c->cfg.batch; hd.capacity = c->cfg.capacity; hd.rebuild_max = c->cfg.rebuild_max;
  hd.max_tokens = c->cfg.max_tokens; hd.ctrl_hidden = c->cfg.ctrl_hidden;
  hd.n = c->n; hd.cur = c->cur; hd.attn = c->attn; hd.step_open = c->step_layer0_done;
  hd.reserved[0] = c->cfg.flags & ADORE_FLAG_RELATIVE_POSITION;   // decides whether the last section is present
  unsigned char* dst = static_cast<unsigned char*>(host_buf);
  std::memset(dst, 0, need);
  std::memcpy(dst, &hd, sizeof(hd));
  size_t off = sizeof(hd);
  for (const StateSection& s : sec) {
    CUDA_OK(cudaMemcpy(dst + off, s.ptr, s.bytes, cudaMemcpyDeviceToHost));
    off += pad8(s.bytes);
  }
  return ADORE_OK;
}

adore_status_t adore_cache_import_state(adore_cache_t* c, const void* host_buf, size_t bytes) {
  if (!c || !host_buf || bytes < sizeof(StateHeader)) return ADORE_ERR_INVALID_ARG;
  StateHeader hd;
  std::memcpy(&hd, host_buf, sizeof(hd));
  const adore_config_t& f = c->cfg;
  if (hd.magic != kStateMagic || hd.version != 1 || hd.batch != f.batch || hd.capacity != f.capacity ||
      hd.rebuild_max != f.rebuild_max || hd.max_tokens != f.max_tokens || hd.ctrl_hidden != f.ctrl_hidden ||
      hd.reserved[0] != (f.flags & ADORE_FLAG_RELATIVE_POSITION) || hd.n < 0 || hd.n > f.max_tokens || (hd.cur != 0 && hd.cur != 1) ||
      (hd.attn != 0 && hd.attn != 1) || hd.step_open < 0 || hd.step_open > 2)
    return ADORE_ERR_INVALID_ARG;
  std::vector<StateSection> sec = state_sections(c);
  add_relative_state(c, sec);
  size_t need = sizeof(StateHeader);
  for (const StateSection& s : sec) need += pad8(s.bytes);
  if (bytes < need) return ADORE_ERR_INVALID_ARG;
  if (!snapshot_consistent(f, hd, static_cast<const unsigned char*>(host_buf), sec)) return ADORE_ERR_INVALID_ARG;
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  if (c->aux && cudaStreamSynchronize(c->aux) != cudaSuccess) return ADORE_ERR_CUDA;
  if (c->ctl && cudaStreamSynchronize(c->ctl) != cudaSuccess) return ADORE_ERR_CUDA;
  const unsigned char* src = static_cast<const unsigned char*>(host_buf);
  size_t off = sizeof(hd);
  for (const StateSection& s : sec) {
    CUDA_OK(cudaMemcpy(s.ptr, src + off, s.bytes, cudaMemcpyHostToDevice));
    off += pad8(s.bytes);
  }
  c->n = hd.n; c->cur = hd.cur; c->attn = hd.attn; c->step_layer0_done = hd.step_open;
  c->joined = true;
  c->rows_gathered = false;
  return ADORE_OK;
}

adore_status_t adore_label_tokens(const float* weights, int32_t n_layers, int32_t batch, int32_t n_heads, int32_t n_slots,
                                  int32_t topk, void* cuda_stream, int32_t* sets, int32_t* count, uint8_t* label,
                                  float* coverage, float* mass) {
  if (!weights || !sets || !count || !label || !coverage || !mass) return ADORE_ERR_INVALID_ARG;
  if (n_layers < 1 || batch < 1 || n_heads < 1 || n_slots < 1 || topk < 2) return ADORE_ERR_INVALID_ARG;
  if (n_slots > kLabelMaxSlots) return ADORE_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int half = topk / 2;
  const size_t smem = size_t(label_pow2(n_slots)) * sizeof(unsigned long long);
  CUDA_OK(cudaMemsetAsync(count, 0, size_t(batch) * n_slots * sizeof(int), st));
  const int n_rows = n_layers * batch * n_heads;
  static const bool full_sort = dev_switch("ADORE_LABELS_FULL_SORT");
  if (!full_sort && half <= kLabelWarpMaxHalf && n_slots <= 32 * kLabelWarpKeysPerLane) {
    int P = 32;
    while (P < half) P <<= 1;
    label_sets_warp_kernel<<<(n_rows + kLabelRowsPerCta - 1) / kLabelRowsPerCta, kLabelThreads,
                             size_t(kLabelRowsPerCta) * P * sizeof(unsigned long long), st>>>(weights, n_rows, batch, n_heads,
                                                                                              n_slots, half, sets, count);
  } else {
    label_sets_kernel<<<n_rows, kLabelThreads, smem, st>>>(weights, batch, n_heads, n_slots, half, sets, count);
  }
  CUDA_OK(cudaGetLastError());
  label_pick_kernel<<<batch, kLabelThreads, smem, st>>>(count, n_slots, topk, label);
  CUDA_OK(cudaGetLastError());
  label_stats_kernel<<<n_layers * batch, kLabelThreads, 0, st>>>(weights, sets, label, batch, n_heads, n_slots, half, coverage, mass);
  CUDA_OK(cudaGetLastError());
  return ADORE_OK;
}

adore_status_t adore_cache_sync_status(adore_cache_t* c) {
  if (!c) return ADORE_ERR_INVALID_ARG;
  if (join_controller(c) != ADORE_OK || join_rebuilds(c) != ADORE_OK) return ADORE_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return ADORE_ERR_CUDA;
  if (c->d2h && cudaStreamSynchronize(c->d2h) != cudaSuccess) return ADORE_ERR_CUDA;   // queued `out` copies
  unsigned word = 0;
  if (cudaMemcpy(&word, c->err, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return ADORE_ERR_CUDA;
  if (word != 0) {
    if (cudaMemset(c->err, 0, sizeof(word)) != cudaSuccess) return ADORE_ERR_CUDA;
    return (word & ERRW_TIMEOUT) ? ADORE_ERR_TIMEOUT : ADORE_ERR_DEVICE_FLAG;
  }
  return ADORE_OK;
}

}  // extern "C"
