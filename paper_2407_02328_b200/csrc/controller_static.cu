// Stateless controller scoring that allocates nothing: the k-split partial sums of the gate
// GEMM, which the cache-based path keeps in a buffer obtained from cudaMalloc at create time,
// live here in a fixed array inside the library image.
#include <cuda_runtime.h>

#include "../../include/adore.h"
#include "controller.cuh"

using namespace adore;

namespace {

// 2 MiB of partial sums: [ksplit][batch][3*d'] doubles. Part of the module image, so every GPU
// that loads the library carries it until the process exits.
constexpr size_t kStaticPartDoubles = 262144;
static __device__ __align__(256) double g_static_part[kStaticPartDoubles];

constexpr int kMaxDevices = 64;
double* g_part_addr[kMaxDevices] = {};      // device address of g_static_part, per device ordinal

// Recurrent half, MLP and score for one token per sequence, reading the matrices in their
// ordinary row-major layout (the cache-based path reads transposed copies; the sums run over
// the same index in the same order).
__global__ void ctrl_score_rowmajor_kernel(const double* part, int ksplit, int B, int h, const float* b_ih,
                                           const float* w_hh, const float* b_hh, const float* pos_w, const float* pos_b,
                                           const float* w1, const float* b1, const float* w2, const float* b2, double* z,
                                           int position, double pos_scale, float* score, float* sigma) {
  extern __shared__ __align__(16) unsigned char smem[];
  double* sm = reinterpret_cast<double*>(smem);
  const int G = 3 * h, tid = threadIdx.x, b = blockIdx.x;
  double* s_z = sm;
  double* s_gi = sm + h;
  double* s_gh = sm + 4 * h;
  double* s_pz = sm + 5 * h;
  double* s_c = sm + 6 * h;
  if (tid < h) s_z[tid] = z[size_t(b) * h + tid];
  __syncthreads();
  if (tid < G) {
    double gi = double(b_ih[tid]);
    for (int ks = 0; ks < ksplit; ++ks) gi += part[(size_t(ks) * B + b) * G + tid];
    double gh = double(b_hh[tid]);
    for (int j = 0; j < h; ++j) gh = fma(double(w_hh[size_t(tid) * h + j]), s_z[j], gh);
    if (tid < 2 * h) s_gi[tid] = gi + gh;
    else { s_gi[tid] = gi; s_gh[tid - 2 * h] = gh; }
  }
  __syncthreads();
  if (tid < h) {
    const double r = 1.0 / (1.0 + exp(-s_gi[tid]));
    const double u = 1.0 / (1.0 + exp(-s_gi[h + tid]));
    const double c = tanh(s_gi[2 * h + tid] + r * s_gh[tid]);
    const double zn = (1.0 - u) * c + u * s_z[tid];
    s_z[tid] = zn;
    s_pz[tid] = double(pos_w[tid]) * (double(position) / pos_scale) + double(pos_b[tid]) + zn;
  }
  __syncthreads();
  double contrib = 0.0;
  if (tid < h) {
    double a = double(b1[tid]);
    for (int j = 0; j < h; ++j) a = fma(double(w1[size_t(tid) * h + j]), s_pz[j], a);
    contrib = double(w2[tid]) * tanh(a);
  }
  contrib = warp_sum(contrib);
  if ((tid & 31) == 0) s_c[tid >> 5] = contrib;
  __syncthreads();
  if (tid == 0) {
    double s = double(b2[0]);
    for (int w = 0; w < (h + 31) / 32; ++w) s += s_c[w];
    score[b] = float(s);
    sigma[b] = float(1.0 / (1.0 + exp(-s)));
  }
  if (tid < h) z[size_t(b) * h + tid] = s_z[tid];
}

}  // namespace

extern "C" adore_status_t adore_controller_score_static(const adore_controller_weights_t* w, adore_dtype_t dtype,
                                                        int32_t batch, int32_t hidden, int32_t ctrl_hidden, const void* x,
                                                        double* z, int32_t position, float pos_scale, float* score,
                                                        float* sigma, void* cuda_stream) {
  if (!w || !x || !z || !score || !sigma || batch < 1 || hidden < 1 || ctrl_hidden < 1 || ctrl_hidden > 256 ||
      position < 0 || !(pos_scale > 0.f) || (dtype != ADORE_F32 && dtype != ADORE_BF16))
    return ADORE_ERR_INVALID_ARG;
  if (!w->gru_w_ih || !w->gru_w_hh || !w->gru_b_ih || !w->gru_b_hh || !w->pos_w || !w->pos_b || !w->mlp_w1 ||
      !w->mlp_b1 || !w->mlp_w2 || !w->mlp_b2)
    return ADORE_ERR_INVALID_ARG;
  // The gate product reads x and W_ih in 16-byte pieces, 32 elements of a row at a time with no bound inside a piece:
  // rows must be whole pieces and start on a 16-byte boundary (the cache-based path has the same rule for `hidden`).
  if (hidden % 64 != 0) return ADORE_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(x) % 16 != 0 || reinterpret_cast<uintptr_t>(w->gru_w_ih) % 16 != 0 ||
      reinterpret_cast<uintptr_t>(z) % 8 != 0)
    return ADORE_ERR_UNSUPPORTED;
  const int G = 3 * ctrl_hidden;
  // the partial sums of one k-slice must fit the fixed array
  if (size_t(batch) * size_t(G) > kStaticPartDoubles) return ADORE_ERR_UNSUPPORTED;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ADORE_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return ADORE_ERR_UNSUPPORTED;
  if (g_part_addr[dev] == nullptr) {
    // first call on this device: the symbol's name is only a host-side handle, kernels need
    // the address it has on the current device
    double* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_part) != cudaSuccess || p == nullptr) {
      cudaGetLastError();
      return ADORE_ERR_CUDA;
    }
    g_part_addr[dev] = p;
  }
  double* part = g_part_addr[dev];
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // split the d-long dot products as far as the array allows (more CTAs for a small batch)
  int ksplit = 1;
  while (ksplit < 16 && size_t(2 * ksplit) * batch * G <= kStaticPartDoubles && hidden / (2 * ksplit) >= kGateKChunk) ksplit *= 2;
  const int per = (hidden + ksplit - 1) / ksplit;
  const int kslice = ((per + kGateKChunk - 1) / kGateKChunk) * kGateKChunk;
  dim3 grid((G + kGateTileG - 1) / kGateTileG, (batch + kGateTileR - 1) / kGateTileR, ksplit);
  if (dtype == ADORE_F32) {
    GateParams<float> g{};
    g.x = static_cast<const float*>(x); g.seq_stride = 1; g.tc = 1; g.rows = batch; g.d = hidden; g.G = G;
    g.w_ih = w->gru_w_ih; g.part = part; g.ksplit = ksplit; g.kslice = kslice;
    ctrl_gates_kernel<float><<<grid, kGateThreads, 0, stream>>>(g);
  } else {
    GateParams<__nv_bfloat16> g{};
    g.x = static_cast<const __nv_bfloat16*>(x); g.seq_stride = 1; g.tc = 1; g.rows = batch; g.d = hidden; g.G = G;
    g.w_ih = w->gru_w_ih; g.part = part; g.ksplit = ksplit; g.kslice = kslice;
    ctrl_gates_kernel<__nv_bfloat16><<<grid, kGateThreads, 0, stream>>>(g);
  }
  if (cudaGetLastError() != cudaSuccess) return ADORE_ERR_CUDA;
  const int threads = G <= 512 ? 512 : 1024;
  ctrl_score_rowmajor_kernel<<<batch, threads, recur_smem_bytes(ctrl_hidden), stream>>>(
      part, ksplit, batch, ctrl_hidden, w->gru_b_ih, w->gru_w_hh, w->gru_b_hh, w->pos_w, w->pos_b, w->mlp_w1, w->mlp_b1,
      w->mlp_w2, w->mlp_b2, z, position, double(pos_scale), score, sigma);
  if (cudaGetLastError() != cudaSuccess) return ADORE_ERR_CUDA;
  return ADORE_OK;
}
