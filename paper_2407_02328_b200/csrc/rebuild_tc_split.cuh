// Rebuild projection for few rows (Section 2.3 with the paper's short lists, R = 8): K split over the two CTAs of a
// thread-block cluster, the halves added through distributed shared memory.
//
// With at most ~150 rows there are fewer 128 x 128 output tiles than half the SMs, and the launch is bound by how fast
// one SM can pull its share of the 67 MB weight matrix. Two CTAs (two SMs) therefore share a tile: CTA r accumulates
// k-blocks [r K/2, (r+1) K/2) in its own tensor memory, exactly like the one-CTA kernel. When both accumulators are
// complete each CTA sends the 64 columns that the OTHER one finishes (CTA 0: columns 0-63, CTA 1: 64-127) into its
// partner's shared memory, the pair meets at a cluster barrier, and each CTA adds part 0 + part 1 for its own 64
// columns and runs the usual epilogue (rotary embedding, bfloat16, scatter) on them. Compared with handing the
// accumulator over through global memory and a counter, nothing waits for a store to become visible device-wide, and
// the epilogue of a tile is shared by two SMs.
//
// Waits: the mbarrier waits are bounded as everywhere (error word + abort flag). The two cluster barriers are reached
// by every thread of both CTAs on every path, also after an abort, so neither CTA can be left waiting.
#pragma once

#include <cooperative_groups.h>

namespace adore {

constexpr int kSplitBN = 128;
constexpr int kSplitHalf = 64;                                   // columns each CTA of the pair finishes
constexpr size_t kSplitXchgBytes = size_t(kSplitHalf) * kTcBM * sizeof(float);   // [64 columns][128 rows]
template <int STAGES>
constexpr size_t split_smem_bytes() { return TcSmem<kSplitBN, STAGES>::kTotal + kSplitXchgBytes; }

__device__ __forceinline__ void split_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void split_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void split_st_remote(uint32_t cluster_addr, float v) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(cluster_addr), "f"(v) : "memory");
}

template <int STAGES>
__global__ void __launch_bounds__(kTcThreads, 1)
rebuild_tc_split_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_w, const TcGemmParams p) {
  namespace cg = cooperative_groups;
  using S = TcSmem<kSplitBN, STAGES>;
  constexpr uint32_t kTmemCols = kSplitBN;
  extern __shared__ __align__(1024) unsigned char tc_smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(tc_smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* tiles = base;
  float* xchg = reinterpret_cast<float*>(base + size_t(STAGES) * S::kStageBytes);          // written by the partner
  uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(STAGES) * S::kStageBytes + kSplitXchgBytes);
  uint64_t* empty = full + STAGES;
  uint64_t* acc_full = empty + STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  cg::cluster_group cluster = cg::this_cluster();
  const uint32_t rank = cluster.block_rank();               // which half of K, and which 64 columns this CTA finishes
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { tc_mbar_init(&full[s], 1u); tc_mbar_init(&empty[s], 1u); }
    tc_mbar_init(acc_full, 1u);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 0) { __syncwarp(); tc_alloc(tmem_slot, kTmemCols); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // first cluster barrier: arrive now, wait just before the first store into the partner's shared memory (by then the
  // partner has long arrived, i.e. it runs)
  split_cluster_arrive();

  wait_for_prior_grid();
  const int M = min(max(*p.row_total - p.row_base, 0), p.row_limit);
  const int m_tiles = (M + kTcBM - 1) / kTcBM, n_tiles = p.N / kSplitBN;
  const int t = int(blockIdx.x >> 1);                       // the pair's tile; the same in both CTAs
  const bool has_tile = t < m_tiles * n_tiles;
  int m0 = 0, n0 = 0;
  if (has_tile) tc_tile_origin<kSplitBN>(t, m_tiles, n_tiles, m0, n0);
  const int k_blocks = p.K / kTcBK;
  const int kb_begin = int(rank) * k_blocks / 2, kb_end = int(rank + 1) * k_blocks / 2;

  if (warp == 0) {
    // ---------------- producer ----------------
    if (lane == 0 && has_tile) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!tc_mbar_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
        unsigned char* sa = tiles + size_t(stage) * S::kStageBytes;
        tc_mbar_expect_tx(&full[stage], uint32_t(S::kStageBytes));
        tc_tma_load_2d(sa, &map_a, kb * kTcBK, m0, &full[stage]);
        tc_tma_load_2d(sa + S::kABytes, &map_w, kb * kTcBK, n0, &full[stage]);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (!ok && !*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
    }
    __syncwarp();
    split_cluster_wait();
    split_cluster_arrive();
    split_cluster_wait();
  } else if (warp == 1) {
    // ---------------- MMA issuer ----------------
    if (lane == 0 && has_tile) {
      constexpr uint32_t idesc = tc_idesc(kTcBM, kSplitBN);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int kb = kb_begin; kb < kb_end; ++kb) {
        if (!tc_mbar_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const unsigned char* sa = tiles + size_t(stage) * S::kStageBytes;
        const uint64_t adesc = tc_smem_desc(sa), bdesc = tc_smem_desc(sa + S::kABytes);
#pragma unroll
        for (int k = 0; k < kTcBK / 16; ++k)
          tc_mma_bf16(tmem_base, adesc + uint64_t(2 * k), bdesc + uint64_t(2 * k), idesc, (kb > kb_begin || k != 0) ? 1u : 0u);
        tc_commit(&empty[stage]);
        if (++stage == STAGES) { stage = 0; phase ^= 1u; }
      }
      if (ok) tc_commit(acc_full);
      else if (!*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
    }
    __syncwarp();
    split_cluster_wait();
    split_cluster_arrive();
    split_cluster_wait();
  } else {
    // ---------------- epilogue (warps 2..5; TMEM lane quarter = warp % 4) ----------------
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const int r = m0 + row_in_tile;
    const bool valid = has_tile && r < M;
    int b = 0, tok = 0, slot = 0;
    if (valid) { b = p.row_b[r]; tok = p.row_tok[r]; slot = p.row_slot[r]; }
    const bool in_range = valid && slot >= 0 && slot < p.C;
    if (valid && !in_range) set_error(p.err, ERRW_BOUNDS);
    const int own0 = n0 + int(rank) * kSplitHalf;             // first of the 64 columns this CTA finishes
    if (in_range) tc_prefetch_rope<kSplitHalf>(p, own0, tok);
    bool ok = has_tile;
    if (ok && !tc_mbar_wait(acc_full, 0u, abort_flag)) {
      ok = false;
      if (lane == 0 && !*abort_flag) { set_error(p.err, ERRW_TIMEOUT); *abort_flag = 1; }
    }
    tc_fence_after();
    ok = __all_sync(0xffffffffu, ok);                        // the TMEM loads below are warp-collective
    split_cluster_wait();                                    // the partner runs: its shared memory may be written
    const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16);
    if (ok) {
      // the 64 columns that the partner finishes go into its exchange buffer, [column][row]: a warp writes 128
      // consecutive bytes per column
      const uint32_t remote = [&] {
        uint32_t a;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(tc_smem_u32(xchg + row_in_tile)), "r"(rank ^ 1u));
        return a;
      }();
#pragma unroll 1
      for (int c = 0; c < kSplitHalf / 32; ++c) {
        uint32_t v[32];
        __syncwarp();
        tc_ld_32x32(taddr + uint32_t(int(rank ^ 1u) * kSplitHalf + c * 32), v);
#pragma unroll
        for (int i = 0; i < 32; ++i) split_st_remote(remote + uint32_t((c * 32 + i) * kTcBM) * 4u, __uint_as_float(v[i]));
      }
    }
    __syncwarp();
    split_cluster_arrive();                                  // release: the stores above are visible to the partner ...
    split_cluster_wait();                                    // ... and its stores to this CTA
    if (ok && !*abort_flag) {
#pragma unroll 1
      for (int c = 0; c < kSplitHalf / 32; ++c) {
        uint32_t v[32];
        __syncwarp();
        tc_ld_32x32(taddr + uint32_t(int(rank) * kSplitHalf + c * 32), v);
        if (in_range) {
          float y[32];
          const float* x = xchg + size_t(c * 32) * kTcBM + row_in_tile;
          // part 0 + part 1 in both CTAs
#pragma unroll
          for (int i = 0; i < 32; ++i)
            y[i] = rank == 0 ? __uint_as_float(v[i]) + x[i * kTcBM] : x[i * kTcBM] + __uint_as_float(v[i]);
          tc_rope_store_32(p, y, own0 + c * 32, b, tok, slot);
        }
      }
    }
  }

  // common exit: TMEM goes back before the CTA ends. Nothing touches the partner's shared memory after the second
  // cluster barrier, so the CTAs may end independently.
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0) { __syncwarp(); tc_dealloc(tmem_base, kTmemCols); }
}

}  // namespace adore
