// Labels for training the controller, and the uniform-token-set statistics (Section 2.2 last paragraph,
// Appendix B "training data collection", Appendix C / Figure 7), from the per-slot attention weights one
// decode step emits for all layers.
//
//   sets[l,b,h]   the K/2 slots with the largest positive weight of that layer and head (descending; equal
//                 weights: lower slot first; -1 padded)
//   count[b,s]    number of those sets that contain slot s
//   label[b,s]    1 for the K slots with the largest positive count (equal counts: lower slot first)
//   coverage[l,b] share of layer l's set members that carry the label
//   mass[l,b]     attention weight of the labelled slots at layer l, averaged over heads
//
// Three kernels: one CTA per (l, b, h) sorts 64-bit keys (weight bits, inverted slot) and counts memberships with
// integer atomics; one CTA per sequence sorts (count, inverted slot); one CTA per (l, b) gathers the statistics.
// Everything integer is exact; `mass` is a float32 sum in a fixed order.
#pragma once

#include "select.cuh"

namespace adore {

constexpr int kLabelThreads = 256;
constexpr int kLabelMaxSlots = 4096;

__host__ __device__ inline int label_pow2(int v) {
  int p = 64;
  while (p < v) p <<= 1;
  return p;
}

// grid = L*B*H
__global__ void __launch_bounds__(kLabelThreads) label_sets_kernel(const float* weights, int B, int H, int S, int half,
                                                                   int* sets, int* count) {
  extern __shared__ __align__(16) unsigned long long lab_keys[];
  const int lbh = blockIdx.x, b = (lbh / H) % B;
  const float* row = weights + size_t(lbh) * S;
  const int P = label_pow2(S);
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    unsigned long long k = 0ull;
    if (i < S) {
      const float w = row[i];
      // positive floats order like their bit patterns; the inverted slot puts the lower slot first among equals
      if (w > 0.f) k = (static_cast<unsigned long long>(__float_as_uint(w)) << 32) | (0xFFFFFFFFu - unsigned(i));
    }
    lab_keys[i] = k;
  }
  __syncthreads();
  bitonic_sort_desc(lab_keys, P);
  for (int j = threadIdx.x; j < half; j += blockDim.x) {
    const unsigned long long k = j < P ? lab_keys[j] : 0ull;
    int slot = -1;
    if (k != 0ull) {
      slot = int(0xFFFFFFFFu - unsigned(k & 0xFFFFFFFFull));
      atomicAdd(&count[size_t(b) * S + slot], 1);
    }
    sets[size_t(lbh) * half + j] = slot;
  }
}

// Same result with one warp per row and no full sort, for K/2 <= 512 and S <= 1056: the row's keys stay in registers,
// the (K/2)-th largest key is found by bisection on the key's bits (a count is a compare, a ballot and a popc; the
// 64-bit keys are all different, so the search ends with exactly K/2 keys at or above the threshold), the kept keys
// are compacted in slot order into shared memory and only those are sorted. grid = ceil(L*B*H / 8), 8 rows per CTA.
constexpr int kLabelRowsPerCta = kLabelThreads / 32;
constexpr int kLabelWarpMaxHalf = 512;
constexpr int kLabelWarpKeysPerLane = 33;

__global__ void __launch_bounds__(kLabelThreads) label_sets_warp_kernel(const float* weights, int n_rows, int B, int H, int S,
                                                                        int half, int* sets, int* count) {
  extern __shared__ __align__(16) unsigned long long lab_keys[];        // [8 warps][pow2 >= half]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int lbh = blockIdx.x * kLabelRowsPerCta + warp;
  if (lbh >= n_rows) return;                                             // whole warps leave; no block barrier below
  const int b = (lbh / H) % B;
  const float* row = weights + size_t(lbh) * S;
  int P = 32;
  while (P < half) P <<= 1;
  unsigned long long* mine = lab_keys + size_t(warp) * P;
  unsigned long long kk[kLabelWarpKeysPerLane];
  int positive = 0;
#pragma unroll
  for (int j = 0; j < kLabelWarpKeysPerLane; ++j) {
    const int i = j * 32 + lane;
    const float w = i < S ? row[i] : 0.f;
    kk[j] = w > 0.f ? ((static_cast<unsigned long long>(__float_as_uint(w)) << 32) | (0xFFFFFFFFu - unsigned(i))) : 0ull;
    positive += __popc(__ballot_sync(0xffffffffu, kk[j] != 0ull));
  }
  unsigned long long thr = 1ull;                                         // fewer than K/2 positive weights: keep them all
  if (positive > half) {
    thr = 0ull;
    for (int bit = 63; bit >= 0; --bit) {
      const unsigned long long cand = thr | (1ull << bit);
      int c = 0;
#pragma unroll
      for (int j = 0; j < kLabelWarpKeysPerLane; ++j) c += __popc(__ballot_sync(0xffffffffu, kk[j] >= cand));
      if (c >= half) thr = cand;
      if (c == half) break;
    }
  }
  // compaction of the kept keys, then a bitonic sort of P keys by this warp alone
  int n_kept = 0;
#pragma unroll
  for (int j = 0; j < kLabelWarpKeysPerLane; ++j) {
    const bool keep = kk[j] >= thr;                                      // thr >= 1: zero keys never pass
    const unsigned m = __ballot_sync(0xffffffffu, keep);
    if (keep) mine[n_kept + __popc(m & ((1u << lane) - 1u))] = kk[j];
    n_kept += __popc(m);
  }
  for (int i = n_kept + lane; i < P; i += 32) mine[i] = 0ull;
  __syncwarp();
  for (int k = 2; k <= P; k <<= 1)
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int t = lane; t < (P >> 1); t += 32) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int l = i | j;
        const unsigned long long a = mine[i], c = mine[l];
        const bool desc = (i & k) == 0;
        if (desc ? (a < c) : (a > c)) { mine[i] = c; mine[l] = a; }
      }
      __syncwarp();
    }
  for (int j = lane; j < half; j += 32) {
    const unsigned long long k = j < P ? mine[j] : 0ull;
    int slot = -1;
    if (k != 0ull) {
      slot = int(0xFFFFFFFFu - unsigned(k & 0xFFFFFFFFull));
      atomicAdd(&count[size_t(b) * S + slot], 1);
    }
    sets[size_t(lbh) * half + j] = slot;
  }
}

// grid = B
__global__ void __launch_bounds__(kLabelThreads) label_pick_kernel(const int* count, int S, int topk, unsigned char* label) {
  extern __shared__ __align__(16) unsigned long long lab_keys[];
  const int b = blockIdx.x;
  const int P = label_pow2(S);
  for (int i = threadIdx.x; i < P; i += blockDim.x) {
    unsigned long long k = 0ull;
    if (i < S) {
      const int c = count[size_t(b) * S + i];
      if (c > 0) k = (static_cast<unsigned long long>(unsigned(c)) << 32) | (0xFFFFFFFFu - unsigned(i));
    }
    lab_keys[i] = k;
  }
  for (int i = threadIdx.x; i < S; i += blockDim.x) label[size_t(b) * S + i] = 0;
  __syncthreads();
  bitonic_sort_desc(lab_keys, P);
  for (int j = threadIdx.x; j < min(topk, P); j += blockDim.x) {
    const unsigned long long k = lab_keys[j];
    if (k != 0ull) label[size_t(b) * S + int(0xFFFFFFFFu - unsigned(k & 0xFFFFFFFFull))] = 1;
  }
}

// grid = L*B
__global__ void __launch_bounds__(kLabelThreads) label_stats_kernel(const float* weights, const int* sets,
                                                                    const unsigned char* label, int B, int H, int S, int half,
                                                                    float* coverage, float* mass) {
  __shared__ int s_int[2][kLabelThreads / 32];
  __shared__ float s_f[kLabelThreads / 32];
  const int lb = blockIdx.x, b = lb % B, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned char* lab = label + size_t(b) * S;
  int members = 0, hit = 0;
  for (int i = tid; i < H * half; i += blockDim.x) {
    const int s = sets[size_t(lb) * H * half + i];
    if (s >= 0) { ++members; hit += lab[s]; }
  }
  // fixed order: thread t adds its elements in ascending index, then a fixed shuffle tree, then warps in order
  float m = 0.f;
  for (int i = tid; i < H * S; i += blockDim.x) {
    const int s = i % S;
    if (lab[s]) m += weights[size_t(lb) * H * S + i];
  }
  for (int o = 16; o > 0; o >>= 1) {
    members += __shfl_xor_sync(0xffffffffu, members, o);
    hit += __shfl_xor_sync(0xffffffffu, hit, o);
    m += __shfl_xor_sync(0xffffffffu, m, o);
  }
  if (lane == 0) { s_int[0][warp] = members; s_int[1][warp] = hit; s_f[warp] = m; }
  __syncthreads();
  if (tid == 0) {
    int mem = 0, h = 0;
    float tot = 0.f;
    for (int w = 0; w < kLabelThreads / 32; ++w) { mem += s_int[0][w]; h += s_int[1][w]; tot += s_f[w]; }
    coverage[lb] = mem > 0 ? float(h) / float(mem) : 0.f;
    mass[lb] = tot / float(H);
  }
}

}  // namespace adore
