// Rebuild projection on the plain ALUs: Y = X_L [W_k ; W_v]^T, rotary embedding, scatter.
//
// Section 2.3: the key/value states of the listed released tokens are recomputed from their
// layer-input rows and written into the freed slots. This variant accumulates in float32 with
// FFMA and is the path of float32 caches (a tensor-core path in tf32 would miss the 1e-4 bound);
// bfloat16 caches use the tcgen05 kernel and keep this one as a cross-check.
#pragma once

#include "common.cuh"

namespace adore {

template <typename T>
struct RebuildParams {
  const T* x_table;       // rows at x_table + (b*seq_stride + tok) * d
  long long seq_stride;
  int d;
  const T* w_kv;          // [N, d], N = 2*H*DH, key rows first
  T* Kc;                  // layer base [B,H,C,DH]
  T* Vc;
  const int* row_b;
  const int* row_tok;
  const int* row_slot;
  const int* row_total;   // device scalar: rows in the whole table
  int row_base;           // this launch covers table rows [row_base, row_base + row_limit) (row_* point at row_base)
  int row_limit;
  const float* rope_cos;  // [max_tokens, DH/2] or nullptr
  const float* rope_sin;
  int H, DH, C, N;
  unsigned* err;
};

constexpr int kSimtTile = 64;
constexpr int kSimtK = 16;

template <typename T>
__global__ void __launch_bounds__(256) rebuild_simt_kernel(const RebuildParams<T> p) {
  __shared__ float As[kSimtK][kSimtTile + 4];
  __shared__ float Ws[kSimtK][kSimtTile + 4];
  __shared__ long long s_rowoff[kSimtTile];
  const int M = min(max(*p.row_total - p.row_base, 0), p.row_limit);
  const int m0 = blockIdx.y * kSimtTile, n0 = blockIdx.x * kSimtTile;
  if (m0 >= M) return;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  if (tid < kSimtTile) {
    const int r = m0 + tid;
    s_rowoff[tid] = r < M ? (static_cast<long long>(p.row_b[r]) * p.seq_stride + p.row_tok[r]) * p.d : -1;
  }
  __syncthreads();
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < p.d; k0 += kSimtK) {
    for (int i = tid; i < kSimtTile * kSimtK; i += 256) {
      const int rr = i / kSimtK, kk = i % kSimtK;
      const long long off = s_rowoff[rr];
      As[kk][rr] = (off >= 0 && k0 + kk < p.d) ? Elem<T>::to_float(p.x_table[off + k0 + kk]) : 0.f;
      const int col = n0 + rr;
      Ws[kk][rr] = (col < p.N && k0 + kk < p.d) ? Elem<T>::to_float(p.w_kv[size_t(col) * p.d + k0 + kk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kSimtK; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; w[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
  const int c0 = n0 + tx * 4;          // four consecutive output columns: two rotary pairs
  if (c0 >= p.N) return;
  const int HD = p.H * p.DH;
  const int part = c0 / HD, h = (c0 % HD) / p.DH, e = c0 % p.DH;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = m0 + ty * 4 + i;
    if (r >= M) continue;
    const int b = p.row_b[r], tok = p.row_tok[r], slot = p.row_slot[r];
    if (slot < 0 || slot >= p.C) { set_error(p.err, ERRW_BOUNDS); continue; }
    float y[4] = {acc[i][0], acc[i][1], acc[i][2], acc[i][3]};
    if (part == 0 && p.rope_cos != nullptr) {
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const float c = p.rope_cos[size_t(tok) * (p.DH / 2) + e / 2 + j];
        const float s = p.rope_sin[size_t(tok) * (p.DH / 2) + e / 2 + j];
        const float a0 = y[2 * j], a1 = y[2 * j + 1];
        y[2 * j] = a0 * c - a1 * s;
        y[2 * j + 1] = a0 * s + a1 * c;
      }
    }
    T* dst = (part == 0 ? p.Kc : p.Vc) + ((size_t(b) * p.H + h) * p.C + slot) * p.DH + e;
#pragma unroll
    for (int j = 0; j < 4; ++j) dst[j] = Elem<T>::from_float(y[j]);
  }
}

}  // namespace adore
