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
#include "mbarrier.cuh"

namespace adore {

constexpr int kGateTileG = 64;     // gates per CTA
constexpr int kGateTileR = 32;     // rows per CTA
constexpr int kGateKChunk = 64;
constexpr int kGateThreads = 256;

template <typename T>
struct GateParams {
  const T* x;            // row r = b*tc + t lives at x + ((b*seq_stride + t) * d); 16-byte aligned rows
  long long seq_stride;  // tokens between consecutive sequences in x
  int tc;                // tokens per sequence in this call
  int rows;              // B * tc
  int d, G;              // input width (multiple of 64), 3*d'
  const float* w_ih;     // [G, d]
  double* part;          // [ksplit + hh_slices, rows, G]
  int ksplit, kslice;    // kslice is a multiple of kGateKInner
  // Decode step only (tc == 1): the recurrent product W_hh z of the same token as hh_slices further k-slices of 64,
  // so that it runs as part of this tiled product (every weight converted once per CTA, shared by all sequences of the
  // tile) instead of once per sequence. CTAs with blockIdx.z >= ksplit take it: k runs over 0 .. h - 1, the weights are
  // w_hh [G, h] and the input row of sequence r is the float64 state z[r, :]. Needs h % 32 == 0.
  int hh_slices, h;
  const float* w_hh;
  const double* z;
};

// 64 gates x 32 rows per CTA, 4 x 2 outputs per thread, float64 FMA, k in chunks of 32. The next
// chunk is fetched into registers while the current one is consumed from shared memory.
constexpr int kGateKInner = 32;
constexpr int kGateHhSlice = 64;   // k-slice of the recurrent product when it rides in the gate product (decode step)

// A decode step's CTA reads a small block of the weight matrix (tile_g rows x a k-slice) through a chain of dependent
// chunk loads, each one round trip to memory; beside a kernel that saturates HBM (the rebuild GEMM) a round trip takes
// several microseconds and the chain was measured at 46 us instead of 14. Asking for the whole block at once (L2
// prefetches, one per 128-byte line, spread over the threads) leaves one such round trip. Blocks above 64 KB (prompt
// chunks, where k is not split) are streamed as before.
__device__ __forceinline__ void gate_prefetch_block(const float* w, int ld, int g0, int tile_g, int G, int k_begin, int k_end) {
  const int cols = k_end - k_begin;
  if (cols <= 0 || size_t(cols) * tile_g * sizeof(float) > 65536) return;
  const int lines = (cols * int(sizeof(float)) + 127) / 128;       // per row; rows start 128-byte aligned when k_begin % 32 == 0
  for (int i = threadIdx.x; i < tile_g * lines; i += blockDim.x) {
    const int g = g0 + i / lines, l = i % lines;
    if (g < G) asm volatile("prefetch.global.L2 [%0];" ::"l"(w + size_t(g) * ld + k_begin + l * 32));
  }
}

template <typename T>
__global__ void __launch_bounds__(kGateThreads) ctrl_gates_kernel(const GateParams<T> p) {
  constexpr int WS = kGateTileG + 2, XS = kGateTileR + 2;       // padded, rows stay 16-byte aligned
  __shared__ __align__(16) double Ws[kGateKInner][WS];
  __shared__ __align__(16) double Xs[kGateKInner][XS];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int g0 = blockIdx.x * kGateTileG, r0 = blockIdx.y * kGateTileR, ks = blockIdx.z;
  let_next_grid_start();                       // a dependent launch may start the part of its work that does not need these sums
  const bool is_hh = ks >= p.ksplit;           // this CTA multiplies the recurrent matrix with the state (decode step)
  const int ld = is_hh ? p.h : p.d;
  const int k_begin = is_hh ? (ks - p.ksplit) * kGateHhSlice : ks * p.kslice;
  const int k_end = is_hh ? min(p.h, k_begin + kGateHhSlice) : min(p.d, k_begin + p.kslice);
  gate_prefetch_block(is_hh ? p.w_hh : p.w_ih, ld, g0, kGateTileG, p.G, k_begin, k_end);
  // per chunk this thread fetches two float4 of W (gates wg, wg+32; k offset 4*wk) and 4 elements of one x row
  const int wk = tid & 7, wg = tid >> 3;
  const int xr = tid >> 3, xk = tid & 7;
  const float* wsrc[2];
  bool wok[2];
#pragma unroll
  for (int j = 0; j < 2; ++j) {
    const int g = g0 + wg + 32 * j;
    wok[j] = g < p.G;
    wsrc[j] = (is_hh ? p.w_hh : p.w_ih) + size_t(wok[j] ? g : 0) * ld + 4 * wk;
  }
  const bool xok = r0 + xr < p.rows;
  const T* xsrc = p.x;
  if (xok) {
    const long long r = r0 + xr, b = r / p.tc, t = r % p.tc;
    xsrc = p.x + (b * p.seq_stride + t) * p.d + 4 * xk;
  }
  float4 wreg[2];
  float xreg[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 2; ++j)
      wreg[j] = wok[j] ? __ldg(reinterpret_cast<const float4*>(wsrc[j] + k0)) : make_float4(0.f, 0.f, 0.f, 0.f);
    if (!xok || is_hh) {                          // (the state is float64: it goes to shared memory directly, below)
      xreg[0] = xreg[1] = xreg[2] = xreg[3] = 0.f;
    } else if (sizeof(T) == 2) {
      const uint2 v = __ldg(reinterpret_cast<const uint2*>(xsrc + k0));
      xreg[0] = __uint_as_float(v.x << 16); xreg[1] = __uint_as_float(v.x & 0xffff0000u);
      xreg[2] = __uint_as_float(v.y << 16); xreg[3] = __uint_as_float(v.y & 0xffff0000u);
    } else {
      const float4 v = __ldg(reinterpret_cast<const float4*>(xsrc + k0));
      xreg[0] = v.x; xreg[1] = v.y; xreg[2] = v.z; xreg[3] = v.w;
    }
  };
  double acc[4][2];
#pragma unroll
  for (int a = 0; a < 4; ++a) { acc[a][0] = 0.0; acc[a][1] = 0.0; }
  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += kGateKInner) {
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int g = wg + 32 * j;
      Ws[4 * wk + 0][g] = double(wreg[j].x);
      Ws[4 * wk + 1][g] = double(wreg[j].y);
      Ws[4 * wk + 2][g] = double(wreg[j].z);
      Ws[4 * wk + 3][g] = double(wreg[j].w);
    }
    if (is_hh) {
#pragma unroll
      for (int e = 0; e < 4; ++e) Xs[4 * xk + e][xr] = xok ? p.z[size_t(r0 + xr) * p.h + k0 + 4 * xk + e] : 0.0;
    } else {
#pragma unroll
      for (int e = 0; e < 4; ++e) Xs[4 * xk + e][xr] = double(xreg[e]);
    }
    __syncthreads();
    if (k0 + kGateKInner < k_end) fetch(k0 + kGateKInner);
#pragma unroll 8
    for (int kk = 0; kk < kGateKInner; ++kk) {
      const double2 wa = *reinterpret_cast<const double2*>(&Ws[kk][2 * tx]);        // gates 2tx, 2tx+1
      const double2 wb = *reinterpret_cast<const double2*>(&Ws[kk][32 + 2 * tx]);   // gates 32+2tx, 33+2tx
      const double2 xv = *reinterpret_cast<const double2*>(&Xs[kk][2 * ty]);
      acc[0][0] = fma(wa.x, xv.x, acc[0][0]); acc[0][1] = fma(wa.x, xv.y, acc[0][1]);
      acc[1][0] = fma(wa.y, xv.x, acc[1][0]); acc[1][1] = fma(wa.y, xv.y, acc[1][1]);
      acc[2][0] = fma(wb.x, xv.x, acc[2][0]); acc[2][1] = fma(wb.x, xv.y, acc[2][1]);
      acc[3][0] = fma(wb.y, xv.x, acc[3][0]); acc[3][1] = fma(wb.y, xv.y, acc[3][1]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int g = g0 + 2 * tx + (a & 1) + 32 * (a >> 1), r = r0 + 2 * ty + c;
      if (g < p.G && r < p.rows) p.part[(size_t(ks) * p.rows + r) * p.G + g] = acc[a][c];
    }
}

// Same product for many rows (prompt chunks, decode at batch >= 48): 128 gates x 64 rows per CTA of 128 threads, 8 x 8
// outputs per thread. Per k the thread reads 8 + 8 operands for 64 FMAs (2 bytes of shared memory per FMA instead of 6
// with the 4 x 2 tile above), which is what the float64 pipe needs to stay busy.
constexpr int kGateWideG = 128;
constexpr int kGateWideR = 64;
constexpr int kGateWideThreads = 128;
constexpr int kGateWideMinRows = 48;     // fewer rows: the 64 x 32 tile kernel wastes less
constexpr int kGateWideWS = kGateWideG + 2, kGateWideXS = kGateWideR + 2;   // padded row lengths (doubles)
constexpr size_t kGateWideSmem = sizeof(double) * kGateKInner * (kGateWideWS + kGateWideXS);

template <typename T>
__global__ void __launch_bounds__(kGateWideThreads) ctrl_gates_wide_kernel(const GateParams<T> p) {
  extern __shared__ __align__(16) double gw_smem[];
  double (*Ws)[kGateWideWS] = reinterpret_cast<double (*)[kGateWideWS]>(gw_smem);
  double (*Xs)[kGateWideXS] = reinterpret_cast<double (*)[kGateWideXS]>(gw_smem + kGateKInner * kGateWideWS);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int g0 = blockIdx.x * kGateWideG, r0 = blockIdx.y * kGateWideR, ks = blockIdx.z;
  let_next_grid_start();
  const bool is_hh = ks >= p.ksplit;           // this CTA multiplies the recurrent matrix with the state (decode step)
  const int ld = is_hh ? p.h : p.d;
  const int k_begin = is_hh ? (ks - p.ksplit) * kGateHhSlice : ks * p.kslice;
  const int k_end = is_hh ? min(p.h, k_begin + kGateHhSlice) : min(p.d, k_begin + p.kslice);
  gate_prefetch_block(is_hh ? p.w_hh : p.w_ih, ld, g0, kGateWideG, p.G, k_begin, k_end);
  // fetch roles: 8 float4 of W (gate (tid + 128 q) / 8, k offset 4 * ((tid + 128 q) % 8)) and 2 x 8 elements of x
  // (row (tid + 128 q) / 4, k offset 8 * ((tid + 128 q) % 4)) per chunk of 32 k
  const float* wsrc[8];
  bool wok[8];
#pragma unroll
  for (int q = 0; q < 8; ++q) {
    const int idx = tid + kGateWideThreads * q, g = g0 + (idx >> 3);
    wok[q] = g < p.G;
    wsrc[q] = (is_hh ? p.w_hh : p.w_ih) + size_t(wok[q] ? g : 0) * ld + 4 * (idx & 7);
  }
  const T* xsrc[2];
  bool xok[2];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int idx = tid + kGateWideThreads * q;
    const long long r = r0 + (idx >> 2);
    xok[q] = r < p.rows;
    xsrc[q] = p.x;
    if (xok[q]) xsrc[q] = p.x + ((r / p.tc) * p.seq_stride + (r % p.tc)) * p.d + 8 * (idx & 3);
  }
  float4 wreg[8];
  float xreg[2][8];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int q = 0; q < 8; ++q)
      wreg[q] = wok[q] ? __ldg(reinterpret_cast<const float4*>(wsrc[q] + k0)) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      if (!xok[q] || is_hh) {                     // (the state is float64: it goes to shared memory directly, below)
#pragma unroll
        for (int e = 0; e < 8; ++e) xreg[q][e] = 0.f;
      } else if (sizeof(T) == 2) {
        const uint4 v = __ldg(reinterpret_cast<const uint4*>(xsrc[q] + k0));
        const uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          xreg[q][2 * e] = __uint_as_float(u[e] << 16);
          xreg[q][2 * e + 1] = __uint_as_float(u[e] & 0xffff0000u);
        }
      } else {
        const float4 a = __ldg(reinterpret_cast<const float4*>(xsrc[q] + k0));
        const float4 b = __ldg(reinterpret_cast<const float4*>(xsrc[q] + k0) + 1);
        xreg[q][0] = a.x; xreg[q][1] = a.y; xreg[q][2] = a.z; xreg[q][3] = a.w;
        xreg[q][4] = b.x; xreg[q][5] = b.y; xreg[q][6] = b.z; xreg[q][7] = b.w;
      }
    }
  };
  double acc[4][4][2][2];       // [gate pair j][row pair i][gate within pair][row within pair]
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i) { acc[j][i][0][0] = acc[j][i][0][1] = acc[j][i][1][0] = acc[j][i][1][1] = 0.0; }
  if (k_begin < k_end) fetch(k_begin);
  for (int k0 = k_begin; k0 < k_end; k0 += kGateKInner) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int idx = tid + kGateWideThreads * q, g = idx >> 3, kk = 4 * (idx & 7);
      Ws[kk + 0][g] = double(wreg[q].x);
      Ws[kk + 1][g] = double(wreg[q].y);
      Ws[kk + 2][g] = double(wreg[q].z);
      Ws[kk + 3][g] = double(wreg[q].w);
    }
#pragma unroll
    for (int q = 0; q < 2; ++q) {
      const int idx = tid + kGateWideThreads * q, r = idx >> 2, kk = 8 * (idx & 3);
      if (is_hh) {
#pragma unroll
        for (int e = 0; e < 8; ++e) Xs[kk + e][r] = xok[q] ? p.z[size_t(r0 + r) * p.h + k0 + kk + e] : 0.0;
      } else {
#pragma unroll
        for (int e = 0; e < 8; ++e) Xs[kk + e][r] = double(xreg[q][e]);
      }
    }
    __syncthreads();
    if (k0 + kGateKInner < k_end) fetch(k0 + kGateKInner);
#pragma unroll 4
    for (int kk = 0; kk < kGateKInner; ++kk) {
      double2 wv[4], xv[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) wv[j] = *reinterpret_cast<const double2*>(&Ws[kk][2 * tx + 32 * j]);
#pragma unroll
      for (int i = 0; i < 4; ++i) xv[i] = *reinterpret_cast<const double2*>(&Xs[kk][2 * ty + 16 * i]);
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[j][i][0][0] = fma(wv[j].x, xv[i].x, acc[j][i][0][0]);
          acc[j][i][0][1] = fma(wv[j].x, xv[i].y, acc[j][i][0][1]);
          acc[j][i][1][0] = fma(wv[j].y, xv[i].x, acc[j][i][1][0]);
          acc[j][i][1][1] = fma(wv[j].y, xv[i].y, acc[j][i][1][1]);
        }
    }
    __syncthreads();
  }
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int a = 0; a < 2; ++a)
#pragma unroll
        for (int b = 0; b < 2; ++b) {
          const int g = g0 + 2 * tx + 32 * j + a, r = r0 + 2 * ty + 16 * i + b;
          if (g < p.G && r < p.rows) p.part[(size_t(ks) * p.rows + r) * p.G + g] = acc[j][i][a][b];
        }
}

struct RecurParams {
  const double* part;    // [ksplit, rows, G], row = b*tc + t; ksplit <= 32 for the prompt kernels, <= 64 for the decode kernel
  int ksplit, rows, tc;
  int h;                 // d'
  const float* b_ih;     // [3h]
  const float* w_hh;     // [3h, h]   recurrent matrix, row-major
  const float* b_hh;     // [3h]
  const float* pos_w;    // [h]
  const float* pos_b;    // [h]
  const float* w1;       // [h, h]    interaction matrix, row-major
  const float* b1;       // [h]
  const float* w2;       // [h]
  const float* b2;       // [1]
  double* z;             // [B, h] state, updated in place
  float* score;          // [B, max_tokens]
  float* sigma;          // [B, max_tokens]
  int max_tokens;
  int n0;                // position of the first token of this call
  double pos_scale;
  int no_recurrence;     // 1: every token sees a zero state (the ablation without the GRU's memory, Section 3.5.3)
  int hh_slices;         // decode kernel: k-slices of `part` after the first ksplit that hold W_hh z (0: it computes that product itself)
  double* a_tab;         // [B, max_tokens, h] or null. Set: positions are relative to the current token; the token is
                         // scored at distance 0 and the input of its Tanh layer is kept for later re-scoring
};


// Shared memory needed by controller_tokens: 7*h + 32 doubles.
__host__ __device__ inline size_t recur_smem_bytes(int h) { return sizeof(double) * (7 * h + 32); }

// Runs p.tc tokens of sequence b through the recurrent half of the GRU and the MLP.
// All threads of the block must call it. Every matrix-vector product is spread over the whole
// block: a warp owns an output row, its lanes split the inner index (coalesced loads that are all
// in flight at once) and a shuffle tree adds the lane partials, in a fixed order.
template <int kCtrlJ>               // inner-index elements per lane: ceil(d' / 32) rounded up to 4 or 8
__device__ __forceinline__ void controller_tokens_impl(const RecurParams& p, int b, double* sm) {
  const int h = p.h, G = 3 * h, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nw = blockDim.x >> 5;
  double* s_z = sm;            // [h]
  double* s_gi = sm + h;       // [3h]  reset/update: input + hidden side; candidate: input side
  double* s_gh = sm + 4 * h;   // [h]   candidate: hidden side
  double* s_pz = sm + 5 * h;   // [h]
  double* s_t = sm + 6 * h;    // [h]   w2[i] * tanh(.)
  if (tid < h) s_z[tid] = p.z[size_t(b) * h + tid];
  __syncthreads();
  for (int t = 0; t < p.tc; ++t) {
    const int row = b * p.tc + t;
    if (p.no_recurrence) {
      __syncthreads();
      for (int i = tid; i < h; i += blockDim.x) s_z[i] = 0.0;
      __syncthreads();
    }
    // four output rows per warp at a time: all their loads are issued before the first is used
    for (int g0 = warp * 4; g0 < G; g0 += nw * 4) {
      float w[4][kCtrlJ];
      double in_part[4];
      float bh[4], bi[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int g = min(g0 + a, G - 1);
#pragma unroll
        for (int jj = 0; jj < kCtrlJ; ++jj) {
          const int j = lane + 32 * jj;
          w[a][jj] = j < h ? __ldg(p.w_hh + size_t(g) * h + j) : 0.f;
        }
        in_part[a] = lane < p.ksplit ? p.part[(size_t(lane) * p.rows + row) * G + g] : 0.0;
        bh[a] = __ldg(p.b_hh + g);
        bi[a] = __ldg(p.b_ih + g);
      }
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int g = g0 + a;
        double acc = 0.0;
#pragma unroll
        for (int jj = 0; jj < kCtrlJ; ++jj) {
          const int j = lane + 32 * jj;
          if (j < h) acc = fma(double(w[a][jj]), s_z[j], acc);
        }
        const double gh = warp_sum(acc) + double(bh[a]);
        const double gi = warp_sum(in_part[a]) + double(bi[a]);
        if (lane == 0 && g < G) {
          if (g < 2 * h) s_gi[g] = gi + gh;
          else { s_gi[g] = gi; s_gh[g - 2 * h] = gh; }
        }
      }
    }
    __syncthreads();
    const int pos = p.n0 + t;
    if (tid < h) {
      const double r = 1.0 / (1.0 + exp(-s_gi[tid]));
      const double u = 1.0 / (1.0 + exp(-s_gi[h + tid]));
      const double c = tanh(s_gi[2 * h + tid] + r * s_gh[tid]);
      const double zn = (1.0 - u) * c + u * s_z[tid];
      s_z[tid] = zn;
      const double upos = p.a_tab ? 0.0 : double(pos) / p.pos_scale;
      s_pz[tid] = double(p.pos_w[tid]) * upos + double(p.pos_b[tid]) + zn;
    }
    __syncthreads();
    for (int i0 = warp * 4; i0 < h; i0 += nw * 4) {
      float w[4][kCtrlJ];
      float bb[4], ww[4];
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int i = min(i0 + a, h - 1);
#pragma unroll
        for (int jj = 0; jj < kCtrlJ; ++jj) {
          const int j = lane + 32 * jj;
          w[a][jj] = j < h ? __ldg(p.w1 + size_t(i) * h + j) : 0.f;
        }
        bb[a] = __ldg(p.b1 + i);
        ww[a] = __ldg(p.w2 + i);
      }
#pragma unroll
      for (int a = 0; a < 4; ++a) {
        const int i = i0 + a;
        double acc = 0.0;
#pragma unroll
        for (int jj = 0; jj < kCtrlJ; ++jj) {
          const int j = lane + 32 * jj;
          if (j < h) acc = fma(double(w[a][jj]), s_pz[j], acc);
        }
        acc = warp_sum(acc);
        if (lane == 0 && i < h) {
          const double pre = acc + double(bb[a]);
          s_t[i] = double(ww[a]) * tanh(pre);
          if (p.a_tab) p.a_tab[(size_t(b) * p.max_tokens + pos) * h + i] = pre;
        }
      }
    }
    __syncthreads();
    if (warp == 0) {
      double acc = 0.0;
      for (int i = lane; i < h; i += 32) acc += s_t[i];
      acc = warp_sum(acc);
      if (lane == 0) {
        const double sc = acc + double(p.b2[0]);
        p.score[size_t(b) * p.max_tokens + pos] = float(sc);
        p.sigma[size_t(b) * p.max_tokens + pos] = float(1.0 / (1.0 + exp(-sc)));
      }
    }
    __syncthreads();
  }
  if (tid < h) p.z[size_t(b) * h + tid] = s_z[tid];
}

// ---- variant with the recurrent matrix resident in shared memory ---------------------------------
// For d' <= 128 (and a multiple of 4) the whole recurrent matrix (3 d' x d' floats, 192 KB at d' = 128)
// fits in shared memory: one elected thread fetches it with bulk copies while the other parameters
// are loaded, the interaction matrix lives in registers (each warp owns d'/16 of its rows), and
// every token then costs only shared-memory reads. This is what makes a long prompt scan cheap and
// takes the weight-load latency off the decode step.
constexpr int kCtrlWarps = 16;                 // the resident variant runs with 512 threads

__host__ __device__ inline bool ctrl_resident_ok(int h) { return h <= 128 && h % 4 == 0; }
// shared memory: matrix | 13h doubles (state, gate sums, input sums) | 8h floats (small vectors) | barrier
__host__ __device__ inline size_t ctrl_resident_smem_bytes(int h) {
  return size_t(3) * h * h * sizeof(float) + sizeof(double) * (13 * h + 32) + sizeof(float) * 8 * h + 16;
}

__device__ __forceinline__ void controller_tokens_resident(const RecurParams& p, int b, unsigned char* smem, unsigned* err) {
  const int h = p.h, G = 3 * h, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  float* s_w = reinterpret_cast<float*>(smem);                    // [3h][h]
  double* sd = reinterpret_cast<double*>(smem + size_t(G) * h * sizeof(float));
  double* s_z = sd;             // [h]
  double* s_gi = sd + h;        // [3h]
  double* s_gh = sd + 4 * h;    // [h]
  double* s_pz = sd + 5 * h;    // [h]
  double* s_t = sd + 6 * h;     // [h]
  double* s_gin = sd + 7 * h;   // [3h] input-side sums (+ bias) of the current token
  float* sf = reinterpret_cast<float*>(sd + 13 * h + 32);
  float* s_bhh = sf;            // [3h]
  float* s_posw = sf + 3 * h;   // [h]
  float* s_posb = sf + 4 * h;   // [h]
  float* s_b1 = sf + 5 * h;     // [h]
  float* s_w2 = sf + 6 * h;     // [h]
  uint64_t* bar = reinterpret_cast<uint64_t*>(sf + 8 * h);

  if (tid == 0) {
    mbar_init(bar, 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    const uint32_t total = uint32_t(G) * h * sizeof(float);
    mbar_expect_tx(bar, total);
    for (uint32_t off = 0; off < total; off += 65536u)
      bulk_g2s(smem + off, reinterpret_cast<const unsigned char*>(p.w_hh) + off, min(65536u, total - off), bar);
  }
  // the interaction matrix in registers: warp w owns rows w*RW .. w*RW+RW-1, lane l columns l, l+32, ...
  constexpr int RW = 8, JN = 4;
  const int rw = (h + kCtrlWarps - 1) / kCtrlWarps;               // rows per warp actually used (<= RW)
  float w1r[RW][JN];
#pragma unroll
  for (int a = 0; a < RW; ++a) {
    const int i = warp * rw + a;
#pragma unroll
    for (int jj = 0; jj < JN; ++jj) {
      const int j = lane + 32 * jj;
      w1r[a][jj] = (a < rw && i < h && j < h) ? __ldg(p.w1 + size_t(i) * h + j) : 0.f;
    }
  }
  for (int i = tid; i < G; i += blockDim.x) s_bhh[i] = p.b_hh[i];
  for (int i = tid; i < h; i += blockDim.x) {
    s_posw[i] = p.pos_w[i]; s_posb[i] = p.pos_b[i]; s_b1[i] = p.b1[i]; s_w2[i] = p.w2[i];
    s_z[i] = p.z[size_t(b) * h + i];
  }
  const float b2 = __ldg(p.b2);
  __syncthreads();
  bool have_w = false;
  for (int t = 0; t < p.tc; ++t) {
    const int row = b * p.tc + t;
    if (p.no_recurrence) {
      __syncthreads();
      for (int i = tid; i < h; i += blockDim.x) s_z[i] = 0.0;
      __syncthreads();
    }
    // input-side sums: the k-slices are added in a fixed order
    for (int g = tid; g < G; g += blockDim.x) {
      double gi = double(__ldg(p.b_ih + g));
#pragma unroll 4
      for (int ks = 0; ks < p.ksplit; ++ks) gi += p.part[(size_t(ks) * p.rows + row) * G + g];
      s_gin[g] = gi;
    }
    if (!have_w) {                                  // first token: the matrix must have landed
      if (!mbar_wait_bounded(bar, 0u, kWaitPolls) && tid == 0) set_error(err, ERRW_TIMEOUT);
      have_w = true;
    }
    __syncthreads();
    // recurrent half: a warp per gate row, a lane per four columns
    {
      double z4[4] = {0.0, 0.0, 0.0, 0.0};
      const int j0 = lane * 4;
      if (j0 < h) { z4[0] = s_z[j0]; z4[1] = s_z[j0 + 1]; z4[2] = s_z[j0 + 2]; z4[3] = s_z[j0 + 3]; }
      // eight rows at a time, so that their shuffle reductions overlap instead of queueing up
      for (int gb = warp; gb < G; gb += kCtrlWarps * 8) {
        double acc[8];
#pragma unroll
        for (int a = 0; a < 8; ++a) {
          const int g = gb + a * kCtrlWarps;
          acc[a] = 0.0;
          if (g < G && j0 < h) {
            const float4 w4 = *reinterpret_cast<const float4*>(s_w + size_t(g) * h + j0);
            acc[a] = fma(double(w4.x), z4[0], acc[a]);
            acc[a] = fma(double(w4.y), z4[1], acc[a]);
            acc[a] = fma(double(w4.z), z4[2], acc[a]);
            acc[a] = fma(double(w4.w), z4[3], acc[a]);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1)
#pragma unroll
          for (int a = 0; a < 8; ++a) acc[a] += __shfl_xor_sync(0xffffffffu, acc[a], o);
        if (lane == 0) {
#pragma unroll
          for (int a = 0; a < 8; ++a) {
            const int g = gb + a * kCtrlWarps;
            if (g < G) {
              const double gh = acc[a] + double(s_bhh[g]);
              if (g < 2 * h) s_gi[g] = s_gin[g] + gh;
              else { s_gi[g] = s_gin[g]; s_gh[g - 2 * h] = gh; }
            }
          }
        }
      }
    }
    __syncthreads();
    const int pos = p.n0 + t;
    if (tid < h) {
      const double r = 1.0 / (1.0 + exp(-s_gi[tid]));
      const double u = 1.0 / (1.0 + exp(-s_gi[h + tid]));
      const double c = tanh(s_gi[2 * h + tid] + r * s_gh[tid]);
      const double zn = (1.0 - u) * c + u * s_z[tid];
      s_z[tid] = zn;
      s_pz[tid] = double(s_posw[tid]) * (p.a_tab ? 0.0 : double(pos) / p.pos_scale) + double(s_posb[tid]) + zn;
    }
    __syncthreads();
    {
      double pz[JN];
#pragma unroll
      for (int jj = 0; jj < JN; ++jj) pz[jj] = (lane + 32 * jj < h) ? s_pz[lane + 32 * jj] : 0.0;
      double acc[RW];
#pragma unroll
      for (int a = 0; a < RW; ++a) {
        acc[a] = 0.0;
#pragma unroll
        for (int jj = 0; jj < JN; ++jj) acc[a] = fma(double(w1r[a][jj]), pz[jj], acc[a]);
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1)
#pragma unroll
        for (int a = 0; a < RW; ++a) acc[a] += __shfl_xor_sync(0xffffffffu, acc[a], o);
      // the tanh of the eight rows is spread over eight lanes
      if (lane < RW) {
        double mine = acc[0];
#pragma unroll
        for (int a = 1; a < RW; ++a) if (lane == a) mine = acc[a];
        const int i = warp * rw + lane;
        if (lane < rw && i < h) {
          const double pre = mine + double(s_b1[i]);
          s_t[i] = double(s_w2[i]) * tanh(pre);
          if (p.a_tab) p.a_tab[(size_t(b) * p.max_tokens + pos) * h + i] = pre;
        }
      }
    }
    __syncthreads();
    if (warp == 0) {
      double acc = 0.0;
      for (int i = lane; i < h; i += 32) acc += s_t[i];
      acc = warp_sum(acc);
      if (lane == 0) {
        const double sc = acc + double(b2);
        p.score[size_t(b) * p.max_tokens + pos] = float(sc);
        p.sigma[size_t(b) * p.max_tokens + pos] = float(1.0 / (1.0 + exp(-sc)));
      }
    }
    __syncthreads();
  }
  if (tid < h) p.z[size_t(b) * h + tid] = s_z[tid];
}

// ---- decode step: one new token per sequence, small footprint ---------------------------------------
// The controller of token n runs beside the attention of layer 0, whose CTAs fill the SMs. The prompt kernel above keeps
// the whole recurrent matrix in shared memory (right for a scan of thousands of tokens), so one CTA needs an SM to itself
// and has to wait until an SM has drained. For the single token of a decode step the recurrent product W_hh z rides in the
// tiled gate product (GateParams::hh_slices) and this kernel does the rest per sequence: it adds the k-slices, applies
// the gates, updates z and runs the two small layers of the MLP. It needs 14 d' doubles of shared memory and shares SMs
// with whatever else is running. Its rows of the interaction matrix are fetched into registers first, so that their
// latency overlaps the k-slice sums. Every sum runs over the same indices in a fixed order (reproducible; float64 as
// everywhere in the controller).
constexpr int kTailThreads = 512;
constexpr int kTailWarps = kTailThreads / 32;
constexpr int kTailRows = 8;                    // matrix rows a warp has in flight

__host__ __device__ inline size_t ctrl_tail_smem_bytes(int h) { return sizeof(double) * (14 * size_t(h) + 32); }

// Rows r0 .. r0 + kTailRows - 1 of a row-major [n_rows, h] float matrix (h % 4 == 0) into registers: lane l takes
// columns 4 l .. 4 l + 3 (and 128 + 4 l .. for h > 128) with 16-byte loads, all of them in flight at once.
__device__ __forceinline__ void tail_rows_load(const float* __restrict__ W, int n_rows, int h, int r0, int lane,
                                               float4 (&w)[kTailRows][2]) {
#pragma unroll
  for (int a = 0; a < kTailRows; ++a) {
    const int r = min(r0 + a, n_rows - 1);
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
      const int j = 4 * lane + 128 * jj;
      w[a][jj] = j < h ? __ldg(reinterpret_cast<const float4*>(W + size_t(r) * h + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
}
// y[a] = sum_j w[a][j] v[j]: the lane's columns, then a shuffle tree over the lanes. Results in every lane.
__device__ __forceinline__ void tail_rows_dot(const float4 (&w)[kTailRows][2], const double (&v)[2][4], double (&y)[kTailRows]) {
#pragma unroll
  for (int a = 0; a < kTailRows; ++a) {
    double acc = 0.0;
#pragma unroll
    for (int jj = 0; jj < 2; ++jj) {
      acc = fma(double(w[a][jj].x), v[jj][0], acc);
      acc = fma(double(w[a][jj].y), v[jj][1], acc);
      acc = fma(double(w[a][jj].z), v[jj][2], acc);
      acc = fma(double(w[a][jj].w), v[jj][3], acc);
    }
    y[a] = acc;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1)
#pragma unroll
    for (int a = 0; a < kTailRows; ++a) y[a] += __shfl_xor_sync(0xffffffffu, y[a], o);
}
// this lane's columns of a shared-memory vector of length h, in the layout of tail_rows_load
__device__ __forceinline__ void tail_lane_columns(const double* s_v, int h, int lane, double (&v)[2][4]) {
#pragma unroll
  for (int jj = 0; jj < 2; ++jj)
#pragma unroll
    for (int e = 0; e < 4; ++e) { const int j = 4 * lane + 128 * jj + e; v[jj][e] = j < h ? s_v[j] : 0.0; }
}
// sum of part[i * stride] for i = i_begin .. i_end - 1, ascending, 24 loads in flight at a time
__device__ __forceinline__ double tail_sum_slices(const double* __restrict__ part, size_t stride, int i_begin, int i_end) {
  double acc = 0.0;
  for (int i0 = i_begin; i0 < i_end; i0 += 24) {
    double t[24];
#pragma unroll
    for (int i = 0; i < 24; ++i) t[i] = i0 + i < i_end ? part[size_t(i0 + i) * stride] : 0.0;
#pragma unroll
    for (int i = 0; i < 24; ++i) acc += t[i];
  }
  return acc;
}

// grid = B CTAs; p.tc must be 1, p.rows = B and p.h a multiple of 4. p.part holds ksplit partial sums of W_ih x per
// (sequence, gate), followed by hh_slices partial sums of W_hh z (hh_slices == 0: the recurrent product is done here).
static __global__ void __launch_bounds__(kTailThreads) ctrl_decode_tail_kernel(const RecurParams p) {
  extern __shared__ __align__(16) unsigned char tail_smem[];
  double* sm = reinterpret_cast<double*>(tail_smem);
  const int h = p.h, G = 3 * h, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, b = blockIdx.x;
  double* s_z = sm;            // [h]
  double* s_gi = sm + h;       // [3h]  input side of every gate (+ bias)
  double* s_gh = sm + 4 * h;   // [3h]  hidden side of every gate (+ bias)
  double* s_pz = sm + 7 * h;   // [h]
  double* s_half = sm + 8 * h; // [2][3h] the two halves of the k-slice sums
  double* s_t = s_gi;          // [h]   w2[i] * tanh(.), reuses the gate sums once they are consumed
  let_next_grid_start();
  // ---- independent of the gate product: the state, this warp's rows of the interaction matrix, and the recurrent half if
  // the gate product does not carry it ----
  for (int i = tid; i < h; i += kTailThreads) s_z[i] = p.no_recurrence ? 0.0 : p.z[size_t(b) * h + i];
  float4 w1r[kTailRows][2];
  const bool mlp_once = h <= kTailWarps * kTailRows;            // every warp has its rows of W1 in registers (d' <= 128)
  if (mlp_once) tail_rows_load(p.w1, h, h, warp * kTailRows, lane, w1r);
  __syncthreads();
  if (p.hh_slices == 0 && !p.no_recurrence) {
    double v[2][4];
    tail_lane_columns(s_z, h, lane, v);
    for (int g0 = warp * kTailRows; g0 < G; g0 += kTailWarps * kTailRows) {
      float4 w[kTailRows][2];
      double y[kTailRows];
      tail_rows_load(p.w_hh, G, h, g0, lane, w);
      tail_rows_dot(w, v, y);
      if (lane < kTailRows && g0 + lane < G) {
        double mine = y[0];
#pragma unroll
        for (int a = 1; a < kTailRows; ++a) if (lane == a) mine = y[a];
        s_gh[g0 + lane] = mine + double(__ldg(p.b_hh + g0 + lane));
      }
    }
  }
  // ---- the k-slices of the input-side product: two threads per gate, each adds one half of the slices in ascending
  // order; then first half + second half ----
  wait_for_prior_grid();
  {
    const size_t stride = size_t(p.rows) * G;
    const int mid = (p.ksplit + 1) / 2;
    for (int item = tid; item < 2 * G; item += kTailThreads) {
      const int g = item % G, half = item / G;
      s_half[half * G + g] = tail_sum_slices(p.part + size_t(b) * G + g, stride, half ? mid : 0, half ? p.ksplit : mid);
    }
    if (p.hh_slices > 0 || p.no_recurrence)
      for (int g = tid; g < G; g += kTailThreads)
        s_gh[g] = double(__ldg(p.b_hh + g)) +
                  (p.no_recurrence ? 0.0 : tail_sum_slices(p.part + size_t(b) * G + g, stride, p.ksplit, p.ksplit + p.hh_slices));
  }
  __syncthreads();
  for (int g = tid; g < G; g += kTailThreads) s_gi[g] = double(__ldg(p.b_ih + g)) + (s_half[g] + s_half[G + g]);
  __syncthreads();
  const int pos = p.n0;
  for (int i = tid; i < h; i += kTailThreads) {
    const double r = 1.0 / (1.0 + exp(-(s_gi[i] + s_gh[i])));
    const double u = 1.0 / (1.0 + exp(-(s_gi[h + i] + s_gh[h + i])));
    const double c = tanh(s_gi[2 * h + i] + r * s_gh[2 * h + i]);
    const double zn = (1.0 - u) * c + u * s_z[i];
    p.z[size_t(b) * h + i] = zn;
    const double upos = p.a_tab ? 0.0 : double(pos) / p.pos_scale;
    s_pz[i] = double(p.pos_w[i]) * upos + double(p.pos_b[i]) + zn;
  }
  __syncthreads();
  {
    double v[2][4];
    tail_lane_columns(s_pz, h, lane, v);
    for (int i0 = warp * kTailRows; i0 < h; i0 += kTailWarps * kTailRows) {
      double y[kTailRows];
      if (!mlp_once) tail_rows_load(p.w1, h, h, i0, lane, w1r);
      tail_rows_dot(w1r, v, y);
      if (lane < kTailRows && i0 + lane < h) {
        double mine = y[0];
#pragma unroll
        for (int a = 1; a < kTailRows; ++a) if (lane == a) mine = y[a];
        const int i = i0 + lane;
        const double pre = mine + double(__ldg(p.b1 + i));
        s_t[i] = double(__ldg(p.w2 + i)) * tanh(pre);
        if (p.a_tab) p.a_tab[(size_t(b) * p.max_tokens + pos) * h + i] = pre;
      }
    }
  }
  __syncthreads();
  if (warp == 0) {
    double acc = 0.0;
    for (int i = lane; i < h; i += 32) acc += s_t[i];
    acc = warp_sum(acc);
    if (lane == 0) {
      const double sc = acc + double(p.b2[0]);
      p.score[size_t(b) * p.max_tokens + pos] = float(sc);
      p.sigma[size_t(b) * p.max_tokens + pos] = float(1.0 / (1.0 + exp(-sc)));
    }
  }
}

// ---- relative positions: every earlier token scored anew at every step ---------------------------
// Section 1 and Figure 2 describe the controller's importance as taken with respect to the token being decoded,
// over all earlier tokens, cached or released. With the position feature read as the distance to the current
// token, u = (n - i) / pos_scale, the score of token i at step n is
//   w2 . tanh(W1 (pos_w u + pos_b + z_i) + b1) + b2  =  w2 . tanh(a_i + u c) + b2,
// with a_i = W1 (pos_b + z_i) + b1 kept from the step the token arrived in (a_tab above) and c = W1 pos_w
// computed once. A step then costs d' tanh per token instead of a d' x d' product, in float64 like the rest of
// the controller (the score decides which token leaves the cache).
struct RescoreParams {
  const double* a_tab;   // [B, max_tokens, h]
  const double* c_vec;   // [h]  W1 pos_w
  const float* w2;       // [h]
  const float* b2;       // [1]
  float* score;          // [B, max_tokens]
  float* sigma;          // [B, max_tokens]
  int h, max_tokens;
  int n;                 // current token; tokens 0 .. n-1 are re-scored
  double pos_scale;
};

constexpr int kRescoreThreads = 256;
constexpr int kRescoreTokens = 32;     // per CTA: one warp per token, four rounds

// c[i] = sum_j W1[i][j] pos_w[j], j ascending. One thread per row; runs once per cache.
static __global__ void ctrl_position_direction_kernel(const float* __restrict__ w1, const float* __restrict__ pos_w, double* c_vec, int h) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= h) return;
  double acc = 0.0;
  for (int j = 0; j < h; ++j) acc = fma(double(w1[size_t(i) * h + j]), double(pos_w[j]), acc);
  c_vec[i] = acc;
}

// grid (ceil(n / kRescoreTokens), B). A warp owns a token: lanes split the d' terms, a shuffle tree adds them in a
// fixed order.
static __global__ void __launch_bounds__(kRescoreThreads) ctrl_rescore_kernel(const RescoreParams p) {
  const int b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  constexpr int kWarps = kRescoreThreads / 32;
  constexpr int JMAX = 8;                      // d' <= 256
  double cj[JMAX];
  float wj[JMAX];
#pragma unroll
  for (int jj = 0; jj < JMAX; ++jj) {
    const int j = lane + 32 * jj;
    cj[jj] = j < p.h ? p.c_vec[j] : 0.0;
    wj[jj] = j < p.h ? __ldg(p.w2 + j) : 0.f;
  }
  const double b2 = double(__ldg(p.b2));
  for (int k = warp; k < kRescoreTokens; k += kWarps) {
    const int i = blockIdx.x * kRescoreTokens + k;
    if (i >= p.n) break;                       // warp-uniform
    const double u = double(p.n - i) / p.pos_scale;
    const double* a = p.a_tab + (size_t(b) * p.max_tokens + i) * p.h;
    double acc = 0.0;
#pragma unroll
    for (int jj = 0; jj < JMAX; ++jj) {
      const int j = lane + 32 * jj;
      if (j < p.h) acc += double(wj[jj]) * tanh(fma(u, cj[jj], a[j]));
    }
    acc = warp_sum(acc);
    if (lane == 0) {
      const double sc = acc + b2;
      p.score[size_t(b) * p.max_tokens + i] = float(sc);
      p.sigma[size_t(b) * p.max_tokens + i] = float(1.0 / (1.0 + exp(-sc)));
    }
  }
}

__device__ inline void controller_tokens(const RecurParams& p, int b, double* sm) {
  if (p.h <= 128) controller_tokens_impl<4>(p, b, sm);
  else controller_tokens_impl<8>(p, b, sm);
}

}  // namespace adore
