// Rebuild projection with the tensor cores of two SMs working on one tile (tcgen05 cta_group::2).
//
// Same contraction and epilogue as rebuild_tc_kernel (Section 2.3: rows of the rebuild list times
// [W_k ; W_v]^T, rotary embedding on the key half, bf16 rounding, scatter into the slots). Two CTAs of a
// cluster share a 256 x 256 output tile: CTA r of the pair stages rows [128 r, 128 r + 128) of the A tile
// and rows [128 r, 128 r + 128) of the W tile (= output columns), the pair's first CTA issues one MMA
// of M = 256, N = 256 per 16 elements of K that reads both CTAs' shared memory, and each CTA's tensor
// memory receives its own 128 rows of the 256-column accumulator. Per SM this halves the W bytes that are
// staged and read per MMA, which is what limits the one-CTA kernel (shared-memory bandwidth shared between
// the TMA writes and the MMA reads).
//
// Barriers (all mbarriers, every wait bounded by wall time):
//   full[s]      in the first CTA: counts the bytes of both CTAs' loads of stage s (the second CTA's TMA
//                signals the first CTA's barrier; no multicast load is used)
//   empty[s]     in both CTAs: tcgen05.commit of the issuing thread arrives on both (stage reusable)
//   acc_full[a]  in both CTAs: same mechanism, accumulator a complete
//   acc_empty[a] in the first CTA: the 4 epilogue warps of each CTA arrive (8 arrivals)
// On a timeout a CTA sets the error bit, raises its own and its partner's abort flag, and every role leaves
// through the common exit; the pair then meets at a cluster barrier and frees its tensor memory.
#pragma once

#include <cooperative_groups.h>

namespace adore {

constexpr int kPairStages = 6;
constexpr int kPairBN = 256;                         // columns of the pair's tile
constexpr int kPairHalfBytes = kTcBM * kTcBK * 2;    // 128 rows x 64 bf16: the A tile and the W half alike
constexpr int kPairStageBytes = 2 * kPairHalfBytes;
constexpr size_t kPairSmemBytes = size_t(kPairStages) * kPairStageBytes + 256 + 1024;

__device__ __forceinline__ uint32_t pair_map_to_cta(uint32_t smem_addr, uint32_t cta_rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
  return r;
}
// TMA tile load whose completion bytes are counted by a barrier that may live in the partner CTA
__device__ __forceinline__ void pair_tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(tc_smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void pair_mbar_arrive_remote(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void pair_alloc(uint32_t* smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(smem_dst)), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void pair_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// arrives (once the MMAs issued so far have completed) on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void pair_commit_both(uint64_t* bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(tc_smem_u32(bar)), "h"(mask) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T with M = 256 (128 rows from each CTA) and N = 256 (128 W rows from each CTA)
__device__ __forceinline__ void pair_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1)
rebuild_tc_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const TcGemmParams p) {
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  constexpr int kStages = kPairStages;
  constexpr int BN = kPairBN;
  constexpr uint32_t kTmemCols = 2 * BN;                  // two accumulators of 256 fp32 columns (128 lanes per CTA)
  extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
  // the dynamic window starts at the same offset in both CTAs, so the rounded base does too
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* tiles = base;
  uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(kStages) * kPairStageBytes);
  uint64_t* empty = full + kStages;
  uint64_t* acc_full = empty + kStages;
  uint64_t* acc_empty = acc_full + 2;
  uint64_t* drained = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drained + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster.block_rank();             // 0: issues the MMAs, owns full[] and acc_empty[]
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  volatile int* partner_abort = cluster.map_shared_rank(const_cast<int*>(abort_flag), rank ^ 1u);
  auto give_up = [&]() {                                   // a wait ran out (or the partner's did)
    if (!*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; *partner_abort = 1; }
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { tc_mbar_init(&full[s], 1u); tc_mbar_init(&empty[s], 1u); }
    for (int a = 0; a < 2; ++a) { tc_mbar_init(&acc_full[a], 1u); tc_mbar_init(&acc_empty[a], 8u); }
    tc_mbar_init(drained, 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) { __syncwarp(); pair_alloc(tmem_slot, kTmemCols); }
  tc_fence_before();
  __syncthreads();
  cluster.sync();                                          // both CTAs' barriers exist before anything crosses over
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // barriers and tensor memory are set up; from here on the kernel touches what earlier kernels wrote
  wait_for_prior_grid();
  const int M = min(max(*p.row_total - p.row_base, 0), p.row_limit);
  const int m_tiles = (M + 2 * kTcBM - 1) / (2 * kTcBM), n_tiles = p.N / BN;
  const int total_tiles = m_tiles * n_tiles;
  const int k_blocks = p.K / kTcBK;

  if (warp == 0) {
    // ---------------- producer: this CTA's half of every stage ----------------
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = pair; t < total_tiles && ok; t += n_pairs) {
        int m0, n0;
        tc_tile_origin<BN, 2 * kTcBM>(t, m_tiles, n_tiles, m0, n0);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!tc_mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* sa = tiles + size_t(stage) * kPairStageBytes;
          const uint32_t bar = pair_map_to_cta(tc_smem_u32(&full[stage]), 0u);
          if (rank == 0) tc_mbar_expect_tx(&full[stage], uint32_t(2 * kPairStageBytes));   // both CTAs' bytes
          pair_tma_load_2d(sa, &map_a, kb * kTcBK, m0 + int(rank) * kTcBM, bar);
          pair_tma_load_2d(sa + kPairHalfBytes, &map_w, kb * kTcBK, n0 + int(rank) * (BN / 2), bar);
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) give_up();
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer (first CTA of the pair only) ----------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = tc_idesc(2 * kTcBM, BN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int t = pair; t < total_tiles && ok; t += n_pairs, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = uint32_t(it >> 1) & 1u;
        if (!tc_mbar_wait(&acc_empty[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + uint32_t(acc * BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!tc_mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          tc_fence_after();
          const unsigned char* sa = tiles + size_t(stage) * kPairStageBytes;
          const uint64_t adesc = tc_smem_desc(sa), bdesc = tc_smem_desc(sa + kPairHalfBytes);
#pragma unroll
          for (int k = 0; k < kTcBK / 16; ++k)
            pair_mma_bf16(d_tmem, adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          pair_commit_both(&empty[stage]);          // both producers may refill the stage once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) pair_commit_both(&acc_full[acc]);   // accumulator complete in both CTAs' tensor memory
      }
      if (!ok) {
        // MMAs may still be in flight on both SMs: wait (bounded) for them before anyone frees anything
        give_up();
        pair_commit_both(drained);
        const unsigned long long t0 = tc_now_ns();
        while (!tc_mbar_try(drained, 0u))
          if (tc_now_ns() - t0 > kTcWaitNs) break;
      }
    }
  } else {
    // ---------------- epilogue (warps 2..5; TMEM lane quarter = warp % 4): this CTA's 128 rows ----------------
    const int quarter = warp & 3;
    bool ok = true;
    int it = 0;
    for (int t = pair; t < total_tiles && ok; t += n_pairs, ++it) {
      const int acc = it & 1;
      const uint32_t acc_phase = uint32_t(it >> 1) & 1u;
      int m0, n0;
      tc_tile_origin<BN, 2 * kTcBM>(t, m_tiles, n_tiles, m0, n0);
      const int r = m0 + int(rank) * kTcBM + quarter * 32 + lane;
      const bool valid = r < M;
      int b = 0, tok = 0, slot = 0;
      if (valid) { b = p.row_b[r]; tok = p.row_tok[r]; slot = p.row_slot[r]; }
      const bool in_range = valid && slot >= 0 && slot < p.C;
      if (valid && !in_range) set_error(p.err, ERRW_BOUNDS);
      if (!tc_mbar_wait(&acc_full[acc], acc_phase, abort_flag)) { ok = false; break; }
      tc_fence_after();
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * BN);
      tc_epilogue_row<BN>(p, taddr, n0, in_range, b, tok, slot);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) pair_mbar_arrive_remote(pair_map_to_cta(tc_smem_u32(&acc_empty[acc]), 0u));
    }
    if (!ok && lane == 0) give_up();
  }

  // common exit: both CTAs arrive here (also after an abort); nothing of the pair is freed before both are done
  tc_fence_before();
  __syncthreads();
  cluster.sync();
  tc_fence_after();
  if (warp == 0) { __syncwarp(); pair_dealloc(tmem_base, kTmemCols); }
}

}  // namespace adore
