// Split-slot decode attention for launches with few (sequence, head) pairs.
//
// Section 2.1 target attention with the top-K mask of Section 2.2 (the phases after the logits are
// shared, attention.cuh). With a small batch there are fewer (b, h) blocks than SMs and one CTA per block leaves
// most of the memory system idle, so a thread-block cluster of S CTAs shares one (b, h):
//   phase 1   CTA r computes the logits of slots [r*C/S, (r+1)*C/S) (the last CTA also takes the
//             current token's own key);
//   exchange  every CTA copies the other CTAs' logits out of their shared memory (distributed shared
//             memory), so that each holds all C+1 logits;
//   phase 2-3 every CTA finds the K-th largest logit and the softmax weights redundantly (identical
//             inputs, identical results; only CTA 0 writes the weights out);
//   phase 4   CTA r accumulates its contiguous share of the kept value rows;
//   reduce    the partial outputs go to CTA 0's shared memory, which adds them, writes `out` and
//             appends the current token's row.
// Only cluster barriers are used for the hand-overs (no spinning on flags).
#pragma once

#include <cooperative_groups.h>

#include "attention.cuh"

namespace adore {

constexpr int kSplitMax = 8;

__host__ __device__ inline size_t attn_split_smem_bytes(int C, int DH) {
  return attn_smem_bytes(C, DH) + sizeof(float) * kSplitMax * DH;
}

template <typename T, int DH>
__global__ void __launch_bounds__(kAttnThreads) attention_split_kernel(const AttnParams<T> p) {
  namespace cg = cooperative_groups;
  constexpr int NT = kAttnThreads;
  constexpr int NW = NT / 32;
  constexpr int EPL = Elem<T>::kPer16B;
  constexpr int LPR = DH / EPL;
  constexpr int RPW = 32 / LPR;
  constexpr int U = kAttnUnroll;

  cg::cluster_group cluster = cg::this_cluster();
  const int S = int(cluster.num_blocks()), rank = int(cluster.block_rank());

  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int C = p.C, rows = C + 1;
  const AttnSmem<DH> sm(smem_raw, rows);
  float* s_logit = sm.logit;
  float* s_parts = reinterpret_cast<float*>(smem_raw + attn_smem_bytes(C, DH));   // [S][DH], used on CTA 0

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, li = lane % LPR;
  const int bh = blockIdx.x / S, b = bh / p.H;
  const size_t row_bytes = size_t(DH) * sizeof(T);
  const unsigned char* Kb = reinterpret_cast<const unsigned char*>(p.Kc) + size_t(bh) * C * row_bytes;
  const unsigned char* knew = reinterpret_cast<const unsigned char*>(p.k_new) + size_t(bh) * row_bytes;
  const int* map = p.slot_tok + size_t(b) * C;
  const int per = (C + S - 1) / S;
  const int lo = min(C, rank * per), hi = (rank == S - 1) ? rows : min(C, lo + per);   // the last CTA owns row C too

  // ---- phase 1: logits of this CTA's rows ----
  float qf[EPL];
  {
    const uint4 qr = *reinterpret_cast<const uint4*>(
        reinterpret_cast<const unsigned char*>(p.q) + size_t(bh) * row_bytes + li * 16);
    Elem<T>::unpack(qr, qf);
  }
  // this CTA's slice of the map row goes to shared memory first (the kept-list area is free until phase 2): a lookup in
  // global memory in front of every key row's load would put two dependent loads in a row
  for (int i = lo + tid; i < min(hi, C); i += NT) sm.list[i] = map[i];
  __syncthreads();
  for (int r0 = lo + warp * RPW; r0 < hi; r0 += NW * RPW * U) {
    uint4 kv[U];
    bool ok[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int row = r0 + u * NW * RPW + sub;
      ok[u] = row < hi && (row == C || sm.list[row] >= 0);
      kv[u] = make_uint4(0u, 0u, 0u, 0u);
      if (ok[u]) kv[u] = ldg_stream((row == C ? knew : Kb + size_t(row) * row_bytes) + li * 16);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int row = r0 + u * NW * RPW + sub;
      float kf[EPL];
      Elem<T>::unpack(kv[u], kf);
      float dot = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) dot = fmaf(qf[e], kf[e], dot);
#pragma unroll
      for (int o = LPR / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
      if (li == 0 && row < hi) s_logit[row] = ok[u] ? dot * p.scale : -INFINITY;
    }
  }
  cluster.sync();                                   // every CTA's slice is in its shared memory

  // ---- exchange: fetch the other slices ----
  for (int r = 0; r < S; ++r) {
    if (r == rank) continue;
    const float* remote = cluster.map_shared_rank(s_logit, r);
    const int rlo = min(C, r * per), rhi = (r == S - 1) ? rows : min(C, rlo + per);
    for (int i = rlo + tid; i < rhi; i += NT) s_logit[i] = remote[i];
  }
  cluster.sync();                                   // nobody overwrites its logits before all have read them

  // ---- phases 2-3 on the full set of logits (redundantly in every CTA) ----
  AttnParams<T> q2 = p;
  if (rank != 0) q2.weights = nullptr;
  const int n_kept = attention_keep_and_weights<T, DH>(q2, sm, bh);

  // ---- phase 4: this CTA's contiguous share of the kept rows ----
  const int share = (n_kept + S - 1) / S;
  const int j_lo = min(n_kept, rank * share), j_hi = min(n_kept, j_lo + share);
  float acc[EPL];
#pragma unroll
  for (int e = 0; e < EPL; ++e) acc[e] = 0.f;
  attention_values_direct<T, DH>(p, sm, bh, j_hi, acc, j_lo);
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
  if (sub == 0)
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm.red[warp * DH + li * EPL + e] = acc[e];
  __syncthreads();
  float* parts0 = cluster.map_shared_rank(s_parts, 0);
  for (int e = tid; e < DH; e += NT) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += sm.red[w * DH + e];
    parts0[rank * DH + e] = s;
  }
  cluster.sync();                                   // all partial outputs have arrived on CTA 0
  if (rank != 0) return;
  for (int e = tid; e < DH; e += NT) {
    float s = 0.f;
    for (int r = 0; r < S; ++r) s += s_parts[r * DH + e];
    p.out[size_t(bh) * DH + e] = Elem<T>::from_float(s);
  }
  if (p.admit_slot != nullptr) {
    const int s = p.admit_slot[b];
    if (s >= 0 && s < C) {
      constexpr int V16 = int(sizeof(T)) * DH / 16;
      unsigned char* kd = reinterpret_cast<unsigned char*>(p.Kc) + (size_t(bh) * C + s) * row_bytes;
      unsigned char* vd = reinterpret_cast<unsigned char*>(p.Vc) + (size_t(bh) * C + s) * row_bytes;
      const unsigned char* vnew = reinterpret_cast<const unsigned char*>(p.v_new) + size_t(bh) * row_bytes;
      if (tid < V16) reinterpret_cast<uint4*>(kd)[tid] = reinterpret_cast<const uint4*>(knew)[tid];
      else if (tid < 2 * V16) reinterpret_cast<uint4*>(vd)[tid - V16] = reinterpret_cast<const uint4*>(vnew)[tid - V16];
    } else if (tid == 0) {
      set_error(p.err, ERRW_BOUNDS);
    }
  }
}

// Number of CTAs that share one (b, h): a power of two <= 8 that brings the launch to about four
// CTAs per SM, 1 when there are enough (b, h) pairs already or the slices would get too short.
inline int attn_split_factor(int items, int C, int sms) {
  int s = 1;
  while (s < kSplitMax && items * s * 2 <= 4 * sms && C / (s * 2) >= 32) s *= 2;
  return s;
}

template <typename T, int DH>
inline cudaError_t launch_attention_split_dh(const AttnParams<T>& p, int items, int S, cudaStream_t stream) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(unsigned(items * S));
  cfg.blockDim = dim3(kAttnThreads);
  cfg.dynamicSmemBytes = attn_split_smem_bytes(p.C, DH);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = unsigned(S);
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attention_split_kernel<T, DH>, p);
}

template <typename T>
inline cudaError_t launch_attention_split(const AttnParams<T>& p, int DH, int items, int S, cudaStream_t stream) {
  if (DH == 64) return launch_attention_split_dh<T, 64>(p, items, S, stream);
  return launch_attention_split_dh<T, 128>(p, items, S, stream);
}

}  // namespace adore
