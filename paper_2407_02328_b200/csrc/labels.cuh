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
