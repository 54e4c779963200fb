// Controller scoring (Section 2.2 Eq. 2 and the line after it; layer sizes from Appendix B):
//   z_i = GRU(x_i, z_{i-1}),  sigma_i = Sigmoid(MLP(p_i + z_i)),  p_i = FC(1->d')(i / pos_scale).
//
// The score decides which token leaves the cache, i.e. it decides integers, so it is computed in
// float64 from the float32 parameters and rounded to float32 once, at the end; ranking happens on
// that float32 value. The cost is small (about 1.6 MFLOP per token) next to the attention bytes.
//
// Two kernels: (1) the input-side gate pre-activations W_ih x for a batch of rows, as a small
// k-split float64 GEMM that writes partial sums; (2) per sequence, the recurrent half, the gates,
// the MLP and the score, summing the partials in a fixed order (results are reproducible).
#pragma once

#include "common.cuh"

namespace adore {

constexpr int kGateTile = 32;     // rows x gates per CTA
constexpr int kGateKChunk = 64;
constexpr int kGateThreads = 256;

template <typename T>
struct GateParams {
  const T* x;            // row r = b*tc + t lives at x + ((b*seq_stride + t) * d)
  long long seq_stride;  // tokens between consecutive sequences in x
  int tc;                // tokens per sequence in this call
  int rows;              // B * tc
  int d, G;              // input width, 3*d'
  const float* w_ih;     // [G, d]
  double* part;          // [ksplit, rows, G]
  int ksplit, kslice;    // kslice is a multiple of kGateKChunk
};

template <typename T>
__global__ void __launch_bounds__(kGateThreads) ctrl_gates_kernel(const GateParams<T> p) {
  __shared__ double Ws[kGateTile][kGateKChunk + 1];
  __shared__ double Xs[kGateTile][kGateKChunk + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int g0 = blockIdx.x * kGateTile, r0 = blockIdx.y * kGateTile, ks = blockIdx.z;
  const int k_begin = ks * p.kslice, k_end = min(p.d, k_begin + p.kslice);
  double acc[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
  for (int k0 = k_begin; k0 < k_end; k0 += kGateKChunk) {
    for (int i = tid; i < kGateTile * kGateKChunk; i += kGateThreads) {
      const int rr = i / kGateKChunk, kk = i % kGateKChunk;
      const int k = k0 + kk;
      const int g = g0 + rr, r = r0 + rr;
      Ws[rr][kk] = (g < p.G && k < k_end) ? double(p.w_ih[size_t(g) * p.d + k]) : 0.0;
      double xv = 0.0;
      if (r < p.rows && k < k_end) {
        const long long b = r / p.tc, t = r % p.tc;
        xv = double(Elem<T>::to_float(p.x[(b * p.seq_stride + t) * p.d + k]));
      }
      Xs[rr][kk] = xv;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < kGateKChunk; ++kk) {
      const double w0 = Ws[tx][kk], w1 = Ws[tx + 16][kk];
      const double x0 = Xs[ty][kk], x1 = Xs[ty + 16][kk];
      acc[0][0] = fma(w0, x0, acc[0][0]);
      acc[0][1] = fma(w0, x1, acc[0][1]);
      acc[1][0] = fma(w1, x0, acc[1][0]);
      acc[1][1] = fma(w1, x1, acc[1][1]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 2; ++a)
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int g = g0 + tx + 16 * a, r = r0 + ty + 16 * c;
      if (g < p.G && r < p.rows) p.part[(size_t(ks) * p.rows + r) * p.G + g] = acc[a][c];
    }
}

struct RecurParams {
  const double* part;    // [ksplit, rows, G], row = b*tc + t
  int ksplit, rows, tc;
  int h;                 // d'
  const float* b_ih;     // [3h]
  const float* w_hh_t;   // [h, 3h]   transposed recurrent matrix
  const float* b_hh;     // [3h]
  const float* pos_w;    // [h]
  const float* pos_b;    // [h]
  const float* w1_t;     // [h, h]    transposed interaction matrix
  const float* b1;       // [h]
  const float* w2;       // [h]
  const float* b2;       // [1]
  double* z;             // [B, h] state, updated in place
  float* score;          // [B, max_tokens]
  float* sigma;          // [B, max_tokens]
  int max_tokens;
  int n0;                // position of the first token of this call
  double pos_scale;
};

// Shared memory needed by controller_tokens: 6*h + 32 doubles.
__host__ __device__ inline size_t recur_smem_bytes(int h) { return sizeof(double) * (6 * h + 32); }

// Runs p.tc tokens of sequence b through the recurrent half of the GRU and the MLP.
// All threads of the block must call it; blockDim.x >= 3*h.
__device__ inline void controller_tokens(const RecurParams& p, int b, double* sm) {
  const int h = p.h, G = 3 * h, tid = threadIdx.x;
  double* s_z = sm;            // [h]
  double* s_gi = sm + h;       // [3h]
  double* s_gh = sm + 4 * h;   // [h] only the candidate's hidden-side term is kept apart
  double* s_pz = sm + 5 * h;   // [h]
  double* s_c = sm + 6 * h;    // [32] warp partials
  if (tid < h) s_z[tid] = p.z[size_t(b) * h + tid];
  __syncthreads();
  for (int t = 0; t < p.tc; ++t) {
    const int row = b * p.tc + t;
    if (tid < G) {
      double gi = double(p.b_ih[tid]);
      for (int ks = 0; ks < p.ksplit; ++ks) gi += p.part[(size_t(ks) * p.rows + row) * G + tid];
      double gh = double(p.b_hh[tid]);
      for (int j = 0; j < h; ++j) gh = fma(double(p.w_hh_t[size_t(j) * G + tid]), s_z[j], gh);
      if (tid < 2 * h) s_gi[tid] = gi + gh;          // reset and update gates: sum of both sides
      else { s_gi[tid] = gi; s_gh[tid - 2 * h] = gh; }
    }
    __syncthreads();
    const int pos = p.n0 + t;
    if (tid < h) {
      const double r = 1.0 / (1.0 + exp(-s_gi[tid]));
      const double u = 1.0 / (1.0 + exp(-s_gi[h + tid]));
      const double c = tanh(s_gi[2 * h + tid] + r * s_gh[tid]);
      const double zn = (1.0 - u) * c + u * s_z[tid];
      s_z[tid] = zn;
      const double upos = double(pos) / p.pos_scale;
      s_pz[tid] = double(p.pos_w[tid]) * upos + double(p.pos_b[tid]) + zn;
    }
    __syncthreads();
    double contrib = 0.0;
    if (tid < h) {
      double a = double(p.b1[tid]);
      for (int j = 0; j < h; ++j) a = fma(double(p.w1_t[size_t(j) * h + tid]), s_pz[j], a);
      contrib = double(p.w2[tid]) * tanh(a);
    }
    contrib = warp_sum(contrib);
    if ((tid & 31) == 0) s_c[tid >> 5] = contrib;
    __syncthreads();
    if (tid == 0) {
      double s = double(p.b2[0]);
      for (int w = 0; w < (h + 31) / 32; ++w) s += s_c[w];
      p.score[size_t(b) * p.max_tokens + pos] = float(s);
      p.sigma[size_t(b) * p.max_tokens + pos] = float(1.0 / (1.0 + exp(-s)));
    }
    __syncthreads();
  }
  if (tid < h) p.z[size_t(b) * h + tid] = s_z[tid];
}

}  // namespace adore
