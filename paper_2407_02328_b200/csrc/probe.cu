// Read-bandwidth probe: what the attention kernel's access pattern can reach on this GPU.
//
// The attention kernel streams every key block and then gathers a scattered subset of 256-byte
// value rows. The copy bandwidth usually quoted as "peak" counts reads and writes of one long
// sequential stream; this probe measures the two read patterns on their own, so that the kernel's
// fraction of the copy peak can be put next to what a plain read kernel achieves.
#include <cuda_runtime.h>

#include "../../include/adore.h"

namespace {

// mode 0: every CTA streams whole blocks of block_rows * row_bytes, grid-stride over the blocks.
// mode 1: every CTA reads rows idx*stride_rows ... of its block: `kept` rows spread evenly with a
//         pseudo-random offset (a stand-in for the kept set of a top-K mask).
__global__ void __launch_bounds__(256) probe_read_kernel(const uint4* __restrict__ data, int n_blocks, int block_rows,
                                                         int row_bytes, int kept, int mode, unsigned* sink) {
  unsigned acc = 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int v_per_row = row_bytes / 16;               // 16-byte pieces per row
  const int rows_per_load = 32 / v_per_row;
  const int stride = max(1, block_rows / max(kept, 1));
  for (int blk = blockIdx.x; blk < n_blocks; blk += gridDim.x) {
    const uint4* base = data + size_t(blk) * block_rows * v_per_row;
    if (mode == 0) {
      const int n16 = block_rows * v_per_row;
      for (int i = threadIdx.x; i < n16; i += blockDim.x * 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = i + u * blockDim.x;
          v[u] = j < n16 ? __ldcs(base + j) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
      }
    } else {
      for (int j0 = warp * rows_per_load; j0 < kept; j0 += nw * rows_per_load * 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int j = j0 + u * nw * rows_per_load + lane / v_per_row;
          // row of the j-th kept entry: one per stride of block_rows / kept rows, at a hashed offset inside it
          const unsigned hsh = (unsigned(blk) * 2654435761u) ^ (unsigned(j) * 40503u);
          const int row = min(block_rows - 1, j * stride + int((hsh >> 8) % unsigned(stride)));
          v[u] = j < kept ? __ldcs(base + size_t(row) * v_per_row + lane % v_per_row) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) acc ^= v[u].x ^ v[u].y ^ v[u].z ^ v[u].w;
      }
    }
  }
  if (acc == 0x9e3779b9u) *sink = acc;               // keeps the loads alive
}

}  // namespace

extern "C" adore_status_t adore_probe_read_bandwidth(const void* buffer, int32_t n_blocks, int32_t block_rows,
                                                     int32_t row_bytes, int32_t kept_rows, int32_t gather,
                                                     int32_t ctas, void* scratch4, void* cuda_stream) {
  if (!buffer || !scratch4 || n_blocks < 1 || block_rows < 1 || ctas < 1 || (row_bytes != 128 && row_bytes != 256 && row_bytes != 512) ||
      (gather && (kept_rows < 1 || kept_rows > block_rows)))
    return ADORE_ERR_INVALID_ARG;
  probe_read_kernel<<<ctas, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint4*>(buffer), n_blocks, block_rows, row_bytes, kept_rows, gather ? 1 : 0,
      static_cast<unsigned*>(scratch4));
  return cudaGetLastError() == cudaSuccess ? ADORE_OK : ADORE_ERR_CUDA;
}
