// Decode attention, phase 1 staged through shared memory by the bulk-copy engine (TMA).
//
// Section 2.1 target attention with the top-K mask of Section 2.2 (the phases after the logits are
// shared, attention.cuh); only the way the key rows reach the SM differs. The K block of one (sequence,
// head) is a contiguous C*dh array, so one elected thread streams it in 8 KB chunks with
// cp.async.bulk into a 4-deep ring; an mbarrier per stage counts the bytes. The warps read the
// rows from shared memory (conflict-free 16-byte accesses). This keeps 24-32 KB in flight per
// CTA without spending registers or issue slots on the loads, which is what the HBM roofline
// needs with several CTAs per SM. The kept value rows are gathered with direct loads.
//
// Every wait is bounded: if a stage never fills, the CTA sets the timeout bit of the error word,
// drains what it issued with short waits and finishes with whatever it has (the step is then
// reported as failed by adore_cache_sync_status).
#pragma once

#include <algorithm>

#include "attention.cuh"
#include "mbarrier.cuh"

namespace adore {

__host__ __device__ inline size_t attn_tma_smem_bytes(int C, int DH, int threads, int kRingStages, int kRingChunkBytes) {
  // ring first (needs 128-byte alignment at most), then barriers (up to 8), then the common carve-up
  return size_t(kRingStages) * kRingChunkBytes + 64 + attn_smem_bytes(C, DH, threads);
}

// NT threads per CTA and kRingStages ring stages are chosen per launch: 128 threads / 2 stages put
// 8-10 CTAs on an SM (fewer, shorter waves when there are many (b, h) pairs), 256 threads / 4 stages
// give each pair more threads (better when there are few pairs or very long key blocks).
// MULTI: several query rows per pair (Section 2.3's rebuilt tokens' rows); the plain decode step compiles without any
// of that logic.
template <typename T, int DH, int NT, int kRingStages, int kRingChunkBytes, bool MULTI>
__global__ void __launch_bounds__(NT, NT <= 128 ? 7 : 4) attention_tma_kernel(const AttnParams<T> p) {
  constexpr int NW = NT / 32;
  constexpr int EPL = Elem<T>::kPer16B;
  constexpr int LPR = DH / EPL;
  constexpr int RPW = 32 / LPR;
  constexpr int ROW_BYTES = DH * int(sizeof(T));
  constexpr int CHUNK_ROWS = kRingChunkBytes / ROW_BYTES;
  static_assert(CHUNK_ROWS % (NW * RPW) == 0, "a chunk must be a whole number of block-wide passes");
  static_assert(kRingStages <= 8, "eight barriers are laid out");
  constexpr int PASSES = CHUNK_ROWS / (NW * RPW);

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* ring = smem_raw;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + size_t(kRingStages) * kRingChunkBytes);
  const int C = p.C, rows = C + 1;
  const AttnSmem<DH, NT> sm(smem_raw + size_t(kRingStages) * kRingChunkBytes + 64, rows);
  float* s_logit = sm.logit;
  int* s_fail = sm.sel + 24;               // one word of the broadcast area
  int* s_last = sm.sel + 25;               // highest occupied slot of the sequence (-1: none)

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, li = lane % LPR;
  // item = one query row; with rows_q > 1 the rows of a (b, h) pair sit next to each other in the grid, so that the
  // pair's key and value blocks are fetched from HBM once and served to the other rows out of L2
  const int rows_q = MULTI ? p.rows_q : 1;
  const int item = blockIdx.x, qi = MULTI ? item % rows_q : 0, bh = MULTI ? item / rows_q : item, b = bh / p.H;
  const bool last_row = !MULTI || qi == rows_q - 1;
  const unsigned char* Kb = reinterpret_cast<const unsigned char*>(p.Kc) + size_t(bh) * C * ROW_BYTES;
  const unsigned char* knew = reinterpret_cast<const unsigned char*>(p.k_new) + size_t(bh) * ROW_BYTES;
  const int* map = p.slot_tok + size_t(b) * C;
  const int n_chunks = (C + CHUNK_ROWS - 1) / CHUNK_ROWS;

  // position bound of this query row (plain decode step: everything occupied is visible)
  int q_tok = 0x7fffffff;
  if (MULTI) {
    wait_for_prior_grid();   // the row table comes from an earlier kernel
    q_tok = last_row ? p.n_cur : p.row_tok[size_t(b) * p.r_max + qi];
    if (q_tok < 0) {                                          // padding row: zeros, nothing else
      for (int e = tid; e < DH; e += NT) p.out[size_t(item) * DH + e] = Elem<T>::from_float(0.f);
      if (p.weights) for (int i = tid; i < rows; i += NT) p.weights[size_t(item) * rows + i] = 0.f;
      return;
    }
  }
  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kRingStages; ++s) mbar_init(&full[s], 1u);
    *s_fail = 0;
    *s_last = -1;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  if (!MULTI) wait_for_prior_grid();   // the cache rows, the slot map and q, k, v come from earlier kernels
  auto issue = [&](int chunk) {
    const int stage = chunk % kRingStages;
    const int r0 = chunk * CHUNK_ROWS;
    const uint32_t bytes = uint32_t(min(CHUNK_ROWS, C - r0)) * ROW_BYTES;
    mbar_expect_tx(&full[stage], bytes);
    bulk_g2s(ring + size_t(stage) * kRingChunkBytes, Kb + size_t(r0) * ROW_BYTES, bytes, &full[stage]);
  };
  if (tid == 0)
    for (int c = 0; c < min(kRingStages, n_chunks); ++c) issue(c);
  // Slots are handed out from the lowest index up, so the empty ones form a tail whenever the cache is not full: the
  // key stream stops after the chunk that holds the highest occupied slot (found while the first chunks are on their way).
  {
    int last = -1;
    for (int i = tid; i < C; i += NT) {
      const int t = map[i];
      sm.list[i] = t;                      // the logit loop reads the map row from here (the list area is free until phase 2)
      if (t >= 0) last = i;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) last = max(last, __shfl_xor_sync(0xffffffffu, last, o));
    if (lane == 0 && last >= 0) atomicMax(s_last, last);
  }

  float qf[EPL];
  {
    const uint4 qr = *reinterpret_cast<const uint4*>(
        reinterpret_cast<const unsigned char*>(p.q) + size_t(item) * ROW_BYTES + li * 16);
    Elem<T>::unpack(qr, qf);
  }
  // the current token's own key (row index C) does not go through the ring
  if (warp == NW - 1 && sub == 0) {
    float kf[EPL];
    Elem<T>::unpack(*reinterpret_cast<const uint4*>(knew + li * 16), kf);
    float dot = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu >> (32 - LPR), dot, o);
    if (li == 0) s_logit[C] = last_row ? dot * p.scale : -INFINITY;
  }

  __syncthreads();                                           // s_last and the staged map row are complete
  // chunks already issued are consumed in any case
  const int n_used = max(min(kRingStages, n_chunks), min(n_chunks, (*s_last + CHUNK_ROWS) / CHUNK_ROWS));
  for (int i = n_used * CHUNK_ROWS + tid; i < C; i += NT) s_logit[i] = -INFINITY;   // the empty tail is never loaded
  bool failed = false;
  for (int c = 0; c < n_used; ++c) {
    const int stage = c % kRingStages;
    const uint32_t parity = uint32_t(c / kRingStages) & 1u;
    if (!mbar_wait_bounded(&full[stage], parity, failed ? kDrainPolls : kWaitPolls)) {
      if (!failed) { set_error(p.err, ERRW_TIMEOUT); *s_fail = 1; }
      failed = true;
    }
    const unsigned char* src = ring + size_t(stage) * kRingChunkBytes;
    const int r0 = c * CHUNK_ROWS;
#pragma unroll
    for (int ps = 0; ps < PASSES; ++ps) {
      const int lr = ps * NW * RPW + warp * RPW + sub;      // row inside the chunk
      const int row = r0 + lr;
      bool ok;
      if (MULTI) {
        const int row_tok = row < C ? sm.list[row] : -1;
        ok = row_tok >= 0 && row_tok <= q_tok && row_tok != p.n_cur;
      } else {
        ok = row < C && sm.list[row] >= 0;
      }
      float kf[EPL];
      // rows past C in a ragged last chunk hold stale bytes of an earlier chunk: read, not used
      Elem<T>::unpack(*reinterpret_cast<const uint4*>(src + size_t(lr) * ROW_BYTES + li * 16), kf);
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      if (li == 0 && row < C) s_logit[row] = ok ? dot * p.scale : -INFINITY;
    }
    __syncthreads();                                         // everyone is done with this stage
    failed = failed || (*s_fail != 0);
    if (tid == 0 && !failed && c + kRingStages < n_used) issue(c + kRingStages);
  }
  // (the loop's last __syncthreads also publishes the logits)
  const int n_kept = attention_keep_and_weights<T, DH, NT>(p, sm, item);

  // ---- phase 4: only the kept value rows, gathered with direct 16-byte loads (one bulk copy per
  // 256-byte row was measured slower than the loads: the copy engine's per-operation cost dominates)
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  constexpr int UV = NT <= 128 ? 8 : 4;     // value-row loads in flight per lane: small CTAs have few warps to hide the latency
  attention_values_direct<T, DH, NT, UV>(p, sm, bh, n_kept, acc);
  attention_finish<T, DH, NT>(p, sm, bh, acc, item, last_row);
}

template <typename T>
inline bool attn_tma_usable(int /*C*/, int DH) { return DH == 64 || DH == 128; }

// CTAs per SM that spread `grid` CTAs evenly over the waves the launch needs anyway. With at most `fit` CTAs on an SM
// it takes w = ceil(grid / (sms * fit)) waves; ceil(grid / (sms * w)) CTAs per SM fill every one of them equally,
// where the greedy placement would run a full wave and then a part-empty one with fewer loads in flight per SM
// (2048 CTAs, fit 8: two waves of 7 per SM instead of 8 and 5.8).
inline int attn_balanced_ctas_per_sm(int grid, int sms, int fit) {
  if (fit < 1 || sms < 1) return fit;
  const int waves = (grid + sms * fit - 1) / (sms * fit);
  return std::min(fit, (grid + sms * waves - 1) / (sms * waves));
}

template <typename T, int DH, int NT, int STAGES, int CHUNK, bool MULTI>
inline cudaError_t launch_attention_tma_as(const AttnParams<T>& p, int grid, cudaStream_t stream) {
  size_t smem = attn_tma_smem_bytes(p.C, DH, NT, STAGES, CHUNK);
  constexpr size_t kSmBytes = 228 * 1024, kCtaReserve = 1024;   // shared memory of an SM, and what the system adds to every CTA
  static bool opted_in = false;            // per instantiation; the attribute is per function
  static int sms = 0, fit_smem = -1, fit = 0;
  auto kernel = attention_tma_kernel<T, DH, NT, STAGES, CHUNK, MULTI>;
  if (!opted_in) {
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 120 * 1024);
    if (e != cudaSuccess) return e;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) sms = 0;
    opted_in = true;
  }
  if (fit_smem != int(smem)) {             // resident CTAs per SM at this shared-memory size (registers and threads included)
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&fit, kernel, NT, smem) != cudaSuccess) { cudaGetLastError(); fit = 0; }
    fit_smem = int(smem);
  }
  const int want = attn_balanced_ctas_per_sm(grid, sms, fit);
  if (want >= 1 && want < fit) {
    // the smallest size that keeps a (want + 1)-th CTA off the SM; whatever is left stays free for kernels that run beside
    const size_t pad = (kSmBytes / size_t(want + 1) - kCtaReserve + 128) & ~size_t(127);
    if (pad > smem && pad <= 120 * 1024) smem = pad;
  }
  return launch_dependent(kernel, dim3(grid), dim3(NT), smem, stream, p);
}
template <typename T, int DH, int NT, int STAGES, int CHUNK>
inline cudaError_t launch_attention_tma_cfg(const AttnParams<T>& p, int grid, cudaStream_t stream) {
  return p.rows_q > 1 ? launch_attention_tma_as<T, DH, NT, STAGES, CHUNK, true>(p, grid, stream)
                      : launch_attention_tma_as<T, DH, NT, STAGES, CHUNK, false>(p, grid, stream);
}

// Many (b, h) pairs with key blocks of moderate length: small CTAs; otherwise large ones (measured on the
// capacity x batch sweep: 128 threads win from ~1000 pairs on up to C = 1024, 256 threads elsewhere).
// Ring: 2 x 8 KB for the small CTAs, 4 x 8 KB for the large ones (the same bytes cut into 4 x 4 KB or 8 x 2 KB stages
// were measured no faster, resp. slower: the key pass is bound by the work per row, not by the bytes in flight).
constexpr int kSmallRingStages = 2, kSmallRingChunk = 8192;
constexpr int kLargeRingStages = 4, kLargeRingChunk = 8192;
template <typename T>
inline cudaError_t launch_attention_tma(const AttnParams<T>& p, int DH, int grid, cudaStream_t stream) {
  const bool small_ctas = grid >= 1024 && p.C <= 1024;
  if (DH == 64) {
    if (small_ctas) return launch_attention_tma_cfg<T, 64, 128, kSmallRingStages, kSmallRingChunk>(p, grid, stream);
    return launch_attention_tma_cfg<T, 64, 256, kLargeRingStages, kLargeRingChunk>(p, grid, stream);
  }
  if (small_ctas) return launch_attention_tma_cfg<T, 128, 128, kSmallRingStages, kSmallRingChunk>(p, grid, stream);
  return launch_attention_tma_cfg<T, 128, 256, kLargeRingStages, kLargeRingChunk>(p, grid, stream);
}

}  // namespace adore
