// Rebuild projection on the 5th-generation tensor cores (tcgen05 + TMEM), bfloat16 caches.
//
// Section 2.3: Y = X_L [W_k ; W_v]^T for the M rows of the step's rebuild list, then the rotary
// embedding on the key half at each token's original position, rounding to bfloat16 and the
// scatter of every head's segment into the token's slot. M is only known on the device.
//
// Structure (persistent, one CTA per SM, 192 threads):
//   warp 0   producer: TMA loads of the A tile (128 x 64) and the W tile (BN x 64), 128-byte
//            swizzle, into a ring of shared-memory stages; an mbarrier per stage counts bytes.
//   warp 1   one thread issues tcgen05.mma (M=128, N=BN, K=16, bf16 -> fp32) into one of two
//            TMEM accumulators; tcgen05.commit releases the stage / publishes the accumulator.
//   warps 2-5 epilogue: tcgen05.ld of the accumulator (32 lanes x 32 columns per warp and step),
//            RoPE on adjacent pairs, bf16 rounding, 16-byte stores straight into the cache rows.
// The accumulator is double buffered, so the epilogue of tile i overlaps the MMAs of tile i+1.
// A rows are first gathered into a compact buffer by gather_rows_kernel (plain TMA afterwards).
// No multicast is used anywhere: every CTA fetches its own tiles.
//
// Every mbarrier wait is bounded by wall time; on expiry the CTA sets the timeout bit, raises an
// abort flag that all roles poll, and leaves through the common exit that frees its TMEM.
#pragma once

#include <cuda.h>

#include <algorithm>
#include <cstdlib>
#include <vector>

#include "../../include/adore.h"
#include "rebuild_simt.cuh"

namespace adore {

constexpr int kTcBM = 128;
constexpr int kTcBK = 64;                    // 64 bf16 = 128 bytes = one swizzle atom
constexpr int kTcThreads = 192;
constexpr unsigned long long kTcWaitNs = 1000000000ull;

// ---- PTX wrappers ------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t tc_smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ unsigned long long tc_now_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void tc_mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(tc_smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(tc_smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(tc_smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool tc_mbar_try(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(tc_smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Waits for the phase with the given parity; gives up after kTcWaitNs or when `abort` is raised.
__device__ __forceinline__ bool tc_mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
  if (tc_mbar_try(bar, parity)) return true;
  const unsigned long long t0 = tc_now_ns();
  uint32_t spins = 0;
  while (!tc_mbar_try(bar, parity)) {
    if ((++spins & 63u) == 0u) {
      if (*abort) return false;
      if (tc_now_ns() - t0 > kTcWaitNs) return false;
    }
  }
  return true;
}
__device__ __forceinline__ void tc_tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(tc_smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(tc_smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_alloc(uint32_t* smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(smem_dst)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tc_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(tc_smem_u32(bar)) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulate, M = 128
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) long,
// stored with the 128-byte swizzle: 8-row groups are 1024 bytes apart (stride byte offset), the
// leading byte offset is not used by swizzled K-major layouts. Bits 46-47: descriptor version 1
// (Blackwell); bits 61-63: swizzle mode 2 = 128 bytes.
__device__ __forceinline__ uint64_t tc_smem_desc(const void* tile) {
  const uint64_t addr = tc_smem_u32(tile);
  return ((addr & 0x3FFFFull) >> 4) | (1ull << 16) | ((1024ull >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor of kind::f16: fp32 accumulator (bits 4-5 = 1), A and B bf16 (bits 7-9 and
// 10-12 = 1), both K-major (bits 15, 16 = 0), N/8 in bits 17-22, M/16 in bits 24-28.
__host__ __device__ constexpr uint32_t tc_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(N >> 3) << 17) | (uint32_t(M >> 4) << 24);
}

// ---- gather of the listed rows into a compact A matrix -----------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) gather_rows_kernel(const T* x_table, long long seq_stride, int d, const int* row_b,
                                                          const int* row_tok, const int* row_total, int row_base,
                                                          int row_limit, T* a_out) {
  let_next_grid_start();
  wait_for_prior_grid();
  const int M = min(max(*row_total - row_base, 0), row_limit);
  for (int r = blockIdx.x; r < M; r += gridDim.x) {
    const uint4* src = reinterpret_cast<const uint4*>(x_table + (static_cast<long long>(row_b[r]) * seq_stride + row_tok[r]) * d);
    uint4* dst = reinterpret_cast<uint4*>(a_out + size_t(r) * d);
    for (int i = threadIdx.x; i < int(d * sizeof(T) / 16); i += blockDim.x) dst[i] = src[i];
  }
}

// ---- the GEMM ------------------------------------------------------------------------------------
struct TcGemmParams {
  __nv_bfloat16* Kc;          // layer base [B,H,C,DH]
  __nv_bfloat16* Vc;
  const int* row_b;
  const int* row_tok;
  const int* row_slot;
  const int* row_total;
  int row_base, row_limit;    // rows [row_base, row_base + row_limit) of the table; row_* point at row_base
  const float* rope_cos;      // [max_tokens, DH/2] or nullptr
  const float* rope_sin;
  int H, DH, C, N, K;
  unsigned* err;
  // split of the K dimension over `ksplit` work units per tile (1 = off). Every unit stores its fp32
  // accumulator in `partial`; the unit that arrives last at the tile's counter adds the parts in ascending
  // order (so the sum does not depend on who was last) and runs the epilogue. Nobody waits for anybody.
  int ksplit;
  float* partial;             // [units][BN * 128] floats per CTA-sized accumulator
  unsigned* unit_cnt;         // [tiles (x 2 CTAs of a pair)][4 lane quarters], zero between launches
};

// STAGES: 4 (256-wide tiles) or 6 (128-wide) fill the SM's shared memory; the 128-wide kernel also exists with 3
// stages (97 KB), which leaves room for CTAs of another kernel on the same SM when a small rebuild runs beside the
// attention of the following layers.
constexpr int kTcLeanStages = 3;
template <int BN, int STAGES = (BN == 256 ? 4 : 6)>
struct TcSmem {
  static constexpr int kStages = STAGES;
  static constexpr int kABytes = kTcBM * kTcBK * 2;
  static constexpr int kBBytes = BN * kTcBK * 2;
  static constexpr int kStageBytes = kABytes + kBBytes;
  static constexpr int kBarrierBytes = 256;
  static constexpr size_t kTotal = size_t(kStages) * kStageBytes + kBarrierBytes + 1024;   // + alignment slack
};

// Tile order: the output columns are walked in bands of kTcBandCols weight rows (about 34 MB of W), all
// row tiles inside a band, columns fastest. A band of W then stays L2-resident while the rows stream
// past it once, instead of the whole 67 MB weight matrix being re-read from DRAM for every wave.
constexpr int kTcBandCols = 4096;
template <int BN, int BM = kTcBM>
__device__ __forceinline__ void tc_tile_origin(int t, int m_tiles, int n_tiles, int& m0, int& n0) {
  constexpr int kBand = kTcBandCols / BN;                 // column tiles per band
  const int per_band = m_tiles * kBand;
  const int band = t / per_band, r = t - band * per_band;
  const int width = min(kBand, n_tiles - band * kBand);   // the last band may be narrower
  m0 = (r / width) * BM;
  n0 = (band * kBand + r % width) * BN;
}

// Epilogue of one accumulator for one output row per lane: reads the row's BN fp32 values from TMEM (32 columns
// at a time; `taddr` addresses this warp's lane quarter and the accumulator's first column), applies the rotary
// embedding to the key half, rounds to bf16 and stores each head's segment at the token's slot. Rows with
// in_range == false take part in the warp-collective TMEM loads and store nothing.
// Layout of one stored accumulator (BN columns x 128 rows): [BN/32 chunks][4 lane quarters][32 columns][32 lanes],
// so that the 32 lanes of a warp write and read consecutive floats.
template <int BN>
__device__ __forceinline__ void tc_store_partial(uint32_t taddr, float* dst, int quarter, int lane) {
#pragma unroll 1
  for (int c = 0; c < BN / 32; ++c) {
    uint32_t v[32];
    __syncwarp();
    tc_ld_32x32(taddr + uint32_t(c * 32), v);
    float* d = dst + (size_t(c * 4 + quarter) * 32) * 32 + lane;
#pragma unroll
    for (int i = 0; i < 32; ++i) d[i * 32] = __uint_as_float(v[i]);
  }
}

// 32 consecutive output columns of one row, starting at column col0 of [K | V]: rotary embedding on the key half
// (adjacent pairs, the token's original position), rounding to bfloat16, four 16-byte stores into the token's slot.
__device__ __forceinline__ void tc_rope_store_32(const TcGemmParams& p, float (&y)[32], int col0, int b, int tok, int slot) {
  const int HD = p.H * p.DH;
  const int part = col0 / HD, h = (col0 % HD) / p.DH, e0 = col0 % p.DH;
  if (part == 0 && p.rope_cos != nullptr) {
    const float4* cs = reinterpret_cast<const float4*>(p.rope_cos + size_t(tok) * (p.DH / 2) + e0 / 2);
    const float4* sn = reinterpret_cast<const float4*>(p.rope_sin + size_t(tok) * (p.DH / 2) + e0 / 2);
#pragma unroll
    for (int g = 0; g < 4; ++g) {
      const float4 c4 = __ldg(cs + g), s4 = __ldg(sn + g);
      const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float a0 = y[8 * g + 2 * j], a1 = y[8 * g + 2 * j + 1];
        y[8 * g + 2 * j] = a0 * cc[j] - a1 * ss[j];
        y[8 * g + 2 * j + 1] = a0 * ss[j] + a1 * cc[j];
      }
    }
  }
  __nv_bfloat16* dst = (part == 0 ? p.Kc : p.Vc) + ((size_t(b) * p.H + h) * p.C + slot) * p.DH + e0;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    uint4 o;
    __nv_bfloat162 t0 = __floats2bfloat162_rn(y[8 * g + 0], y[8 * g + 1]);
    __nv_bfloat162 t1 = __floats2bfloat162_rn(y[8 * g + 2], y[8 * g + 3]);
    __nv_bfloat162 t2 = __floats2bfloat162_rn(y[8 * g + 4], y[8 * g + 5]);
    __nv_bfloat162 t3 = __floats2bfloat162_rn(y[8 * g + 6], y[8 * g + 7]);
    o.x = *reinterpret_cast<uint32_t*>(&t0); o.y = *reinterpret_cast<uint32_t*>(&t1);
    o.z = *reinterpret_cast<uint32_t*>(&t2); o.w = *reinterpret_cast<uint32_t*>(&t3);
    reinterpret_cast<uint4*>(dst)[g] = o;
  }
}

// Asks for the lines of a token's rotary table that the key columns [n0, n0 + BN) of its row will read, so that the
// epilogue's loads, issued only when the accumulator is complete, find them in the cache.
template <int BN>
__device__ __forceinline__ void tc_prefetch_rope(const TcGemmParams& p, int n0, int tok) {
  const int HD = p.H * p.DH;
  if (p.rope_cos == nullptr || n0 >= HD) return;            // no rotation, or a value tile
  for (int col = n0; col < min(n0 + BN, HD); col += 64) {   // 64 columns = 32 angles = one 128-byte line of each table
    const size_t at = size_t(tok) * (p.DH / 2) + (col % p.DH) / 2;
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p.rope_cos + at));
    asm volatile("prefetch.global.L1 [%0];" ::"l"(p.rope_sin + at));
  }
}

// `parts` > 1: the row's values are the sum over the stored accumulators parts_base + q * part_stride, q ascending,
// with this unit's own part (`my_part`) taken from TMEM. Two parts: the other unit's 32 values of the NEXT column
// chunk are requested before the current chunk is worked on, so that only the first request's latency shows.
template <int BN>
__device__ __forceinline__ void tc_epilogue_row(const TcGemmParams& p, uint32_t taddr, int n0, bool in_range, int b, int tok,
                                                int slot, int quarter = 0, int lane = 0, int parts = 1, int my_part = 0,
                                                const float* parts_base = nullptr, size_t part_stride = 0) {
  const bool two = parts == 2;
  const float* other = two ? parts_base + size_t(1 - my_part) * part_stride + size_t(quarter) * 1024 + lane : nullptr;
  float nxt[32];
  if (two && in_range) {
#pragma unroll
    for (int i = 0; i < 32; ++i) nxt[i] = __ldcg(other + i * 32);
  }
#pragma unroll 1
  for (int c = 0; c < BN / 32; ++c) {
    uint32_t v[32];
    __syncwarp();                               // the TMEM load is warp-collective
    tc_ld_32x32(taddr + uint32_t(c * 32), v);
    const int col0 = n0 + c * 32;
    if (in_range) {
      float y[32];
      if (two) {
        // part 0 + part 1 whichever unit runs this: the sum does not depend on who arrived last
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = my_part == 0 ? __uint_as_float(v[i]) + nxt[i] : nxt[i] + __uint_as_float(v[i]);
        if (c + 1 < BN / 32) {
          const float* src = other + size_t(c + 1) * 4096;
#pragma unroll
          for (int i = 0; i < 32; ++i) nxt[i] = __ldcg(src + i * 32);
        }
      } else if (parts > 1) {
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = 0.f;
        for (int q = 0; q < parts; ++q) {
          if (q == my_part) {
#pragma unroll
            for (int i = 0; i < 32; ++i) y[i] += __uint_as_float(v[i]);
          } else {
            const float* src = parts_base + size_t(q) * part_stride + (size_t(c * 4 + quarter) * 32) * 32 + lane;
#pragma unroll
            for (int i = 0; i < 32; ++i) y[i] += __ldcg(src + i * 32);
          }
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) y[i] = __uint_as_float(v[i]);
      }
      tc_rope_store_32(p, y, col0, b, tok, slot);
    }
  }
}

// Split-K hand-over for one warp (one lane quarter of one CTA-sized accumulator): stores the accumulator, then
// counts itself in. Returns true for the warp that arrived last; it also puts the counter back to zero.
template <int BN>
__device__ __forceinline__ bool tc_split_arrive(const TcGemmParams& p, uint32_t taddr, float* my_slot, unsigned* cnt,
                                                int quarter, int lane) {
  tc_store_partial<BN>(taddr, my_slot, quarter, lane);
  __threadfence();
  __syncwarp();
  unsigned old = 0;
  if (lane == 0) old = atomicAdd(cnt, 1u);
  old = __shfl_sync(0xffffffffu, old, 0);
  const bool last = old == unsigned(p.ksplit - 1);
  if (last) {
    if (lane == 0) *cnt = 0u;
    __threadfence();
  }
  return last;
}

template <int BN, int STAGES = (BN == 256 ? 4 : 6)>
__global__ void __launch_bounds__(kTcThreads, 1)
rebuild_tc_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const TcGemmParams p) {
  using S = TcSmem<BN, STAGES>;
  constexpr int kStages = S::kStages;
  constexpr uint32_t kTmemCols = 2 * BN;                  // two fp32 accumulators of BN columns
  extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* tiles = base;
  uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(kStages) * S::kStageBytes);
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { tc_mbar_init(&full[s], 1u); tc_mbar_init(&empty[s], 1u); }
    for (int a = 0; a < 2; ++a) { tc_mbar_init(&acc_full[a], 1u); tc_mbar_init(&acc_empty[a], 4u); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) { __syncwarp(); tc_alloc(tmem_slot, kTmemCols); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // barriers and tensor memory are set up; from here on the kernel touches what earlier kernels wrote
  wait_for_prior_grid();
  const int M = min(max(*p.row_total - p.row_base, 0), p.row_limit);
  const int m_tiles = (M + kTcBM - 1) / kTcBM, n_tiles = p.N / BN;
  const int total_tiles = m_tiles * n_tiles * p.ksplit;      // work units: (tile, part of K), parts of a tile adjacent
  const int k_blocks = p.K / kTcBK;

  if (warp == 0) {
    // ---------------- producer ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int u = blockIdx.x; u < total_tiles && ok; u += gridDim.x) {
        const int t = u / p.ksplit, part = u - t * p.ksplit;
        int m0, n0;
        tc_tile_origin<BN>(t, m_tiles, n_tiles, m0, n0);
        const int kb_end = (part + 1) * k_blocks / p.ksplit;
        for (int kb = part * k_blocks / p.ksplit; kb < kb_end; ++kb) {
          if (!tc_mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = tiles + size_t(stage) * S::kStageBytes;
          tc_mbar_expect_tx(&full[stage], uint32_t(S::kStageBytes));
          tc_tma_load_2d(sa, &map_a, kb * kTcBK, m0, &full[stage]);
          tc_tma_load_2d(sa + S::kABytes, &map_w, kb * kTcBK, n0, &full[stage]);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok && !*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0) {
      constexpr uint32_t idesc = tc_idesc(kTcBM, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int u = blockIdx.x; u < total_tiles && ok; u += gridDim.x, ++it) {
        const int part = u % p.ksplit;
        const int acc = it & 1;
        const uint32_t acc_phase = uint32_t(it >> 1) & 1u;
        if (!tc_mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + uint32_t(acc * BN);
        const int kb_begin = part * k_blocks / p.ksplit, kb_end = (part + 1) * k_blocks / p.ksplit;
        for (int kb = kb_begin; kb < kb_end; ++kb) {
          if (!tc_mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const unsigned char* sa = tiles + size_t(stage) * S::kStageBytes;
          const uint64_t adesc = tc_smem_desc(sa), bdesc = tc_smem_desc(sa + S::kABytes);
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k)      // 16 bf16 = 32 bytes further along K: +2 in 16-byte units
            tc_mma_bf16(d_tmem, adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc, (kb > kb_begin || k != 0) ? 1u : 0u);
          tc_commit(&empty[stage]);                 // stage reusable once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) tc_commit(&acc_full[acc]);          // accumulator complete
      }
      if (!ok && !*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // ---------------- epilogue (warps 2..5; TMEM lane quarter = warp % 4) ----------------
    const int quarter = warp & 3;
    bool ok = true;
    int it = 0;
    for (int u = blockIdx.x; u < total_tiles && ok; u += gridDim.x, ++it) {
      const int t = u / p.ksplit, part = u - t * p.ksplit;
      const int acc = it & 1;
      const uint32_t acc_phase = uint32_t(it >> 1) & 1u;
      int m0, n0;
      tc_tile_origin<BN>(t, m_tiles, n_tiles, m0, n0);
      const int r = m0 + quarter * 32 + lane;
      const bool valid = r < M;
      int b = 0, tok = 0, slot = 0;
      if (valid) { b = p.row_b[r]; tok = p.row_tok[r]; slot = p.row_slot[r]; }
      const bool in_range = valid && slot >= 0 && slot < p.C;
      if (valid && !in_range) set_error(p.err, ERRW_BOUNDS);
      if (in_range) tc_prefetch_rope<BN>(p, n0, tok);
      if (!tc_mbar_wait(&acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * BN);
      if (p.ksplit == 1) {
        tc_epilogue_row<BN>(p, taddr, n0, in_range, b, tok, slot);
      } else {
        constexpr size_t kPart = size_t(BN) * 128;
        float* tile_parts = p.partial + size_t(t) * p.ksplit * kPart;
        if (tc_split_arrive<BN>(p, taddr, tile_parts + size_t(part) * kPart, p.unit_cnt + t * 4 + quarter, quarter, lane))
          tc_epilogue_row<BN>(p, taddr, n0, in_range, b, tok, slot, quarter, lane, p.ksplit, part, tile_parts, kPart);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) tc_mbar_arrive(&acc_empty[acc]);   // this warp has drained its quarter
    }
    if (!ok && lane == 0 && !*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
  }

  // common exit: everyone arrives here (also after an abort); TMEM goes back before the CTA ends
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) { __syncwarp(); tc_dealloc(tmem_base, kTmemCols); }
}

}  // namespace adore

#include "rebuild_tc_pair.cuh"   // the two-SM variant of the kernel above (uses its wrappers and epilogue)
#include "rebuild_tc_split.cuh"  // few rows: K split over a pair of CTAs, halves added through distributed shared memory

namespace adore {

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*TcEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  bool ready = false;
  TcEncodeFn encode = nullptr;
  int sms = 148;
  int N = 0, K = 0;
  int pairs = 0;                      // CTA pairs the two-SM kernel runs with (0: not available)
  int split_pairs = 0;                // CTA pairs the K-split kernel can hold at once (0: not available)
  size_t a_rows = 0;                  // rows of the gather buffer (multiple of 256)
  __nv_bfloat16* a_buf = nullptr;
  float* partial = nullptr;           // split-K accumulators: one 128 x 256 fp32 block per SM
  unsigned* unit_cnt = nullptr;       // split-K arrival counters (kTcCounters words, zero between launches)
  CUtensorMap map_a{};
  std::vector<CUtensorMap> map_w256;  // per layer, W tile of 256 rows (only if N % 256 == 0)
  std::vector<CUtensorMap> map_w128;  // per layer, W tile of 128 rows
  std::vector<char> has_w;
};

constexpr int kTcCounters = 4096;
constexpr size_t kTcPartialFloatsPerSm = size_t(256) * 128;

// Which kernel and which split of K serve a launch of at most `rows` rows. Enough 256 x 256 tiles for every SM pair:
// the two-SM kernel (tensor-bound). Enough 128 x 256 tiles for every SM: those. Otherwise the launch is bound by the
// latency of streaming each weight tile once (measured: ~1.5 us per 32 KB stage with six stages in flight, i.e.
// ~0.3 us per k-block whatever the tile), so 128 x 128 tiles, and K split in two when that still leaves SMs idle: over
// the two CTAs of a cluster that add their halves through distributed shared memory (kind 3) where the device can hold
// that many pairs, else over two independent work units that hand over through global memory and a counter (kind 0).
struct TcPlan { int kind; int ksplit; int grid; };   // kind 0: 128-wide tiles, 1: 256-wide tiles, 2: SM pairs, 3: K split over a CTA pair
inline TcPlan tc_plan(int rows, int N, int K, int sms, int pairs, int max_split, int split_pairs = 0) {
  const int kb = K / kTcBK;
  const int mt128 = (rows + kTcBM - 1) / kTcBM, mt256 = (rows + 2 * kTcBM - 1) / (2 * kTcBM);
  if (pairs > 0 && N % 256 == 0 && mt256 * (N / 256) >= pairs) return TcPlan{2, 1, 2 * pairs};
  if (N % 256 == 0 && mt128 * (N / 256) >= sms) return TcPlan{1, 1, sms};
  const int tiles = mt128 * (N / 128);
  const bool split = max_split >= 2 && kb % 2 == 0 && kb / 2 >= 4 && 2 * tiles <= sms && 4 * tiles <= kTcCounters;
  if (split && tiles <= split_pairs) return TcPlan{3, 2, 2 * tiles};
  const int units = split ? 2 * tiles : tiles;
  return TcPlan{0, split ? 2 : 1, std::max(1, std::min(sms, units))};
}

inline bool tc_encode_2d(TcState& s, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {uint32_t(kTcBK), box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return s.encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T> inline bool tc_usable(const TcState&) { return false; }
template <> inline bool tc_usable<__nv_bfloat16>(const TcState& s) { return s.ready; }

inline adore_status_t tc_init(TcState& s, const adore_config_t& f, std::vector<void*>& owned, cudaStream_t) {
  s.N = 2 * f.n_heads * f.head_dim;
  s.K = f.hidden;
  if (s.N % 128 != 0 || s.K % kTcBK != 0) return ADORE_OK;          // shape not tiled: the ALU path serves it
  if (dev_switch("ADORE_REBUILD_SIMT")) return ADORE_OK;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || fn == nullptr ||
      q != cudaDriverEntryPointSuccess)
    return ADORE_ERR_CUDA;
  s.encode = reinterpret_cast<TcEncodeFn>(fn);
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&s.sms, cudaDevAttrMultiProcessorCount, dev);
  const size_t want = size_t(f.batch) * size_t(std::max(f.rebuild_max, std::min(f.capacity, 32768 / std::max(1, f.batch) + 1)));
  const size_t full = size_t(f.batch) * f.capacity;
  s.a_rows = ((std::min(std::max(want, size_t(f.batch) * f.rebuild_max), full) + 2 * kTcBM - 1) / (2 * kTcBM)) * (2 * kTcBM);
  if (s.a_rows < size_t(2 * kTcBM)) s.a_rows = 2 * kTcBM;
  void* ptr = nullptr;
  if (cudaMalloc(&ptr, s.a_rows * s.K * 2) != cudaSuccess) { cudaGetLastError(); return ADORE_ERR_OOM; }
  owned.push_back(ptr);
  s.a_buf = static_cast<__nv_bfloat16*>(ptr);
  if (cudaMemset(ptr, 0, s.a_rows * s.K * 2) != cudaSuccess) return ADORE_ERR_CUDA;
  if (!tc_encode_2d(s, &s.map_a, s.a_buf, s.a_rows, s.K, kTcBM)) return ADORE_ERR_CUDA;
  if (cudaMalloc(&ptr, size_t(s.sms) * kTcPartialFloatsPerSm * sizeof(float)) != cudaSuccess) { cudaGetLastError(); return ADORE_ERR_OOM; }
  owned.push_back(ptr);
  s.partial = static_cast<float*>(ptr);
  if (cudaMalloc(&ptr, kTcCounters * sizeof(unsigned)) != cudaSuccess) { cudaGetLastError(); return ADORE_ERR_OOM; }
  owned.push_back(ptr);
  s.unit_cnt = static_cast<unsigned*>(ptr);
  if (cudaMemset(ptr, 0, kTcCounters * sizeof(unsigned)) != cudaSuccess) return ADORE_ERR_CUDA;
  s.map_w256.resize(f.n_layers);
  s.map_w128.resize(f.n_layers);
  s.has_w.assign(f.n_layers, 0);
  if (cudaFuncSetAttribute(rebuild_tc_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(TcSmem<256>::kTotal)) != cudaSuccess ||
      cudaFuncSetAttribute(rebuild_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(TcSmem<128>::kTotal)) != cudaSuccess ||
      cudaFuncSetAttribute(rebuild_tc_kernel<128, kTcLeanStages>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(TcSmem<128, kTcLeanStages>::kTotal)) != cudaSuccess)
    return ADORE_ERR_CUDA;
  // the two-SM kernel needs pairs of SMs that can host a cluster of two 1-CTA-per-SM blocks
  if (s.N % kPairBN == 0 && !dev_switch("ADORE_REBUILD_ONE_SM") &&
      cudaFuncSetAttribute(rebuild_tc_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(kPairSmemBytes)) == cudaSuccess) {
    cudaLaunchConfig_t lc{};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.gridDim = dim3(unsigned(s.sms / 2 * 2)); lc.blockDim = dim3(kTcThreads); lc.dynamicSmemBytes = kPairSmemBytes;
    lc.attrs = at; lc.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, rebuild_tc_pair_kernel, &lc) == cudaSuccess) s.pairs = std::min(clusters, s.sms / 2);
  }
  cudaGetLastError();
  // the K-split kernel: pairs of SMs again, with its own (larger) shared-memory footprint
  if (cudaFuncSetAttribute(rebuild_tc_split_kernel<6>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(split_smem_bytes<6>())) == cudaSuccess &&
      cudaFuncSetAttribute(rebuild_tc_split_kernel<kTcLeanStages>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           int(split_smem_bytes<kTcLeanStages>())) == cudaSuccess) {
    cudaLaunchConfig_t lc{};
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.gridDim = dim3(unsigned(s.sms / 2 * 2)); lc.blockDim = dim3(kTcThreads); lc.dynamicSmemBytes = split_smem_bytes<6>();
    lc.attrs = at; lc.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, rebuild_tc_split_kernel<6>, &lc) == cudaSuccess) s.split_pairs = std::min(clusters, s.sms / 2);
  }
  cudaGetLastError();
  s.ready = true;
  return ADORE_OK;
}

inline adore_status_t tc_set_weights(TcState& s, int layer, const void* w_kv) {
  if (!s.ready) return ADORE_OK;
  if (s.N % 256 == 0 && !tc_encode_2d(s, &s.map_w256[layer], w_kv, uint64_t(s.N), uint64_t(s.K), 256u)) return ADORE_ERR_CUDA;
  if (!tc_encode_2d(s, &s.map_w128[layer], w_kv, uint64_t(s.N), uint64_t(s.K), 128u)) return ADORE_ERR_CUDA;
  s.has_w[layer] = 1;
  return ADORE_OK;
}

// Gathers the rows and runs the GEMM, in chunks of at most a_rows rows. Returns the launches made.
template <typename T>
inline cudaError_t launch_rebuild_tc(TcState&, const RebuildParams<T>&, int, int, cudaStream_t, int*, bool, bool = false) { return cudaErrorNotSupported; }
template <typename T>
inline cudaError_t launch_gather_tc(TcState&, const RebuildParams<T>&, int, cudaStream_t) { return cudaErrorNotSupported; }

// Gathers rows [0, m_max) of the row table into the compact A buffer (m_max <= a_rows).
template <>
inline cudaError_t launch_gather_tc<__nv_bfloat16>(TcState& s, const RebuildParams<__nv_bfloat16>& rp, int m_max, cudaStream_t stream) {
  const int gather_grid = std::min(m_max, 8 * s.sms);
  return launch_dependent(gather_rows_kernel<__nv_bfloat16>, dim3(gather_grid), dim3(256), 0, stream, rp.x_table, rp.seq_stride,
                          rp.d, rp.row_b, rp.row_tok, rp.row_total, 0, m_max, s.a_buf);
}

template <>
inline cudaError_t launch_rebuild_tc<__nv_bfloat16>(TcState& s, const RebuildParams<__nv_bfloat16>& rp, int layer, int m_max,
                                                    cudaStream_t stream, int* launched, bool rows_in_place, bool lean) {
  // rows_in_place: the A buffer already holds the listed rows (gathered earlier for this row table; one chunk only)
  // lean: the launch runs beside another kernel; a weight-streaming (128-wide) launch then takes the small ring
  *launched = 0;
  if (!s.has_w[layer]) return cudaErrorInvalidValue;
  // the table may hold more rows than the gather buffer: go through it in chunks
  for (int base = 0; base < m_max; base += int(s.a_rows)) {
    const int limit = std::min(m_max - base, int(s.a_rows));
    cudaError_t e = cudaSuccess;
    if (!(rows_in_place && base == 0 && m_max <= int(s.a_rows))) {
      const int gather_grid = std::min(limit, 8 * s.sms);
      e = launch_dependent(gather_rows_kernel<__nv_bfloat16>, dim3(gather_grid), dim3(256), 0, stream, rp.x_table, rp.seq_stride,
                           rp.d, rp.row_b + base, rp.row_tok + base, rp.row_total, base, limit, s.a_buf);
      ++*launched;
      if (e != cudaSuccess) return e;
    }
    TcGemmParams g{};
    g.Kc = rp.Kc; g.Vc = rp.Vc; g.row_b = rp.row_b + base; g.row_tok = rp.row_tok + base; g.row_slot = rp.row_slot + base;
    g.row_total = rp.row_total; g.row_base = base; g.row_limit = limit;
    g.rope_cos = rp.rope_cos; g.rope_sin = rp.rope_sin; g.H = rp.H; g.DH = rp.DH; g.C = rp.C; g.N = rp.N; g.K = rp.d; g.err = rp.err;
    static const int max_split = dev_switch_int("ADORE_TC_KSPLIT_MAX", 4);
    const TcPlan plan = tc_plan(limit, s.N, s.K, s.sms, s.pairs, max_split, s.split_pairs);
    g.ksplit = plan.ksplit; g.partial = s.partial; g.unit_cnt = s.unit_cnt;
    if (plan.kind == 2) {
      cudaLaunchConfig_t lc{};
      cudaLaunchAttribute at[2];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[1].val.programmaticStreamSerializationAllowed = 1;
      static const bool no_dep = dev_switch("ADORE_NO_DEPENDENT_LAUNCH");
      lc.gridDim = dim3(unsigned(plan.grid)); lc.blockDim = dim3(kTcThreads); lc.dynamicSmemBytes = kPairSmemBytes;
      lc.stream = stream; lc.attrs = at; lc.numAttrs = no_dep ? 1 : 2;
      e = cudaLaunchKernelEx(&lc, rebuild_tc_pair_kernel, s.map_a, s.map_w128[layer], g);
      ++*launched;
      if (e != cudaSuccess) return e;
      continue;
    }
    if (plan.kind == 3) {
      cudaLaunchConfig_t lc{};
      // (an ordinary launch: as a programmatic dependent this cluster launch kept the controller's gate product, which
      // runs beside it on another stream, from finishing before the GEMM did: 14 -> 46 us)
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
      lc.gridDim = dim3(unsigned(plan.grid)); lc.blockDim = dim3(kTcThreads); lc.stream = stream; lc.attrs = at; lc.numAttrs = 1;
      if (lean) {
        lc.dynamicSmemBytes = split_smem_bytes<kTcLeanStages>();
        e = cudaLaunchKernelEx(&lc, rebuild_tc_split_kernel<kTcLeanStages>, s.map_a, s.map_w128[layer], g);
      } else {
        lc.dynamicSmemBytes = split_smem_bytes<6>();
        e = cudaLaunchKernelEx(&lc, rebuild_tc_split_kernel<6>, s.map_a, s.map_w128[layer], g);
      }
      ++*launched;
      if (e != cudaSuccess) return e;
      continue;
    }
    if (plan.kind == 1)
      e = launch_dependent(rebuild_tc_kernel<256>, dim3(plan.grid), dim3(kTcThreads), TcSmem<256>::kTotal, stream, s.map_a,
                           s.map_w256[layer], g);
    else if (lean)
      e = launch_dependent(rebuild_tc_kernel<128, kTcLeanStages>, dim3(plan.grid), dim3(kTcThreads),
                           TcSmem<128, kTcLeanStages>::kTotal, stream, s.map_a, s.map_w128[layer], g);
    else
      e = launch_dependent(rebuild_tc_kernel<128>, dim3(plan.grid), dim3(kTcThreads), TcSmem<128>::kTotal, stream, s.map_a,
                           s.map_w128[layer], g);
    ++*launched;
    if (e != cudaSuccess) return e;
  }
  return cudaGetLastError();
}

}  // namespace adore
