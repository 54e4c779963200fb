// Attention of Section 2.3 with several query rows per (sequence, head) on the tensor cores (bfloat16 caches).
//
// The R_max + 1 query rows of a pair (the rebuilt tokens' rows and the current token's; at most 16) share ONE pass
// over the pair's key rows and ONE over its value rows:
//   phase 1  S = Q K^T. The key block streams through shared memory in tiles of 64 rows (TMA, 128-byte swizzle);
//            the 16 x dh query block sits in registers as the A operand of mma.sync.m16n8k16, each of the 8 warps
//            takes 8 keys of a tile (B operand via ldmatrix). Logits go to shared memory, masked by each row's
//            position bound (a row sees tokens up to its own position; the slot reserved for the current token
//            is not written yet and is skipped).
//   phase 2  one warp per row: K-th largest logit by bisection on the bits of an order-preserving key (counting with
//            compares and warp sums, no atomics), softmax, weights in place (and to global memory if asked for).
//   phase 3  O = P V. The value block streams through the same ring; P is split into a bfloat16 head and a
//            bfloat16 remainder (two MMAs per step) so that the weights enter with ~2^-17 relative error;
//            each warp takes one of a tile's four k-steps and half of the output columns, the partial outputs are
//            added through shared memory. The current token's own value row is added for the last row.
// Then the current token's rows are stored in their slot. Every mbarrier wait is bounded.
// More than 16 rows per pair (the paper's range goes to R = 32): the kernel exists with RB = 3 blocks of 16 rows, which
// share every key and value fragment read from shared memory, so that up to 48 rows still take one pass over the pair's
// keys and one over its values (one CTA per SM then: the logits of 48 rows need most of the shared memory). Rows beyond
// what fits go in groups, one launch per group (row_base / rows_total in the parameters); the groups of a pair read its
// key and value blocks again (from L2 when the launches follow one another closely), and only the last group, which
// holds the current token's row, adds that token's own key and value and stores its rows.
#pragma once

#include <cuda.h>

#include "attention.cuh"
#include "mbarrier.cuh"

namespace adore {

constexpr int kRowsThreads = 256;
constexpr int kRowsWarps = kRowsThreads / 32;
constexpr int kRowsTile = 64;            // key / value rows per tile
constexpr int kRowsStages = 4;
constexpr int kRowsMaxQ = 16;            // rows of one block (the M of one MMA)
constexpr int kRowsMaxBlocks = 3;        // row blocks a CTA can carry through one pass
constexpr int kRowsKeysPerLaneMax = 33;  // logits of a row per lane: C + 1 <= 1056

__host__ __device__ inline int rows_logit_stride(int C) {
  int sp = (C + 1 + 3) & ~3;
  if (sp % 32 == 0) sp += 4;
  return sp;
}
__host__ __device__ inline size_t rows_smem_bytes(int C, int DH, int rows_q) {
  return 1024 + size_t(kRowsStages) * kRowsTile * DH * 2 + 64 + sizeof(int) * kRowsMaxQ * kRowsMaxBlocks +
         sizeof(int) * size_t((C + 3) & ~3) +
         sizeof(float) * size_t(rows_q) * rows_logit_stride(C);
}

__device__ __forceinline__ void rows_tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void rows_ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void rows_ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void rows_mma(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t rows_pack_bf16(float lo, float hi) {
  const __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&t);
}
// Byte offset of element (row, 16-byte chunk `c16` of the 128-byte line) inside a 64-row x 128-byte tile stored with the
// 128-byte swizzle (tile base 1024-byte aligned): the chunk index is XORed with the row's low three bits.
__device__ __forceinline__ uint32_t rows_swz(int row, int c16) { return uint32_t(row) * 128u + (uint32_t(c16 ^ (row & 7)) << 4); }

// KPL: logits of a row held per lane during the selection (C + 1 <= 32 KPL); the counting loops run over all KPL
// registers without guards (slots past the row hold key 0, which never counts).
template <int DH, int KPL, int RB>
__global__ void __launch_bounds__(kRowsThreads)
attention_rows_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const AttnParams<__nv_bfloat16> p) {
  using T = __nv_bfloat16;
  constexpr int HALVES = DH / 64;                       // 64-column (128-byte) boxes per tile
  constexpr int TILE_BYTES = kRowsTile * DH * 2;
  constexpr int KSTEPS = DH / 16;
  extern __shared__ __align__(1024) unsigned char rows_smem_raw[];
  unsigned char* base = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(rows_smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* ring = base;
  uint64_t* full = reinterpret_cast<uint64_t*>(base + size_t(kRowsStages) * TILE_BYTES);
  int* s_qtok = reinterpret_cast<int*>(full + 8);       // [48] position bound per row (< 0: padding)
  int* s_tok = s_qtok + kRowsMaxQ * kRowsMaxBlocks;     // [C] the pair's slot map row (token position per slot)
  float* S = reinterpret_cast<float*>(s_tok + ((p.C + 3) & ~3));

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int bh = blockIdx.x, b = bh / p.H;
  const int C = p.C, R1 = p.rows_q, SP = rows_logit_stride(C);
  const int RT = p.rows_total > 0 ? p.rows_total : R1;  // rows per pair in q / out / weights
  const int rb = p.rows_total > 0 ? p.row_base : 0;     // first row of this launch's group
  const bool has_last = rb + R1 == RT;                  // the group ends with the current token's row
  // tiles are consumed two at a time (one block barrier and one round of refills per 128 rows): an even count, the
  // tile past the end, if any, holds rows of the next pair or zeros and is masked like every row >= C
  const int n_tiles = (((C + kRowsTile - 1) / kRowsTile) + 1) & ~1;
  const int* map = p.slot_tok + size_t(b) * C;

  if (tid == 0) {
    for (int s = 0; s < kRowsStages; ++s) mbar_init(&full[s], 1u);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  wait_for_prior_grid();
  if (tid < kRowsMaxQ * RB) {
    const int g = rb + tid;                             // row index within the pair
    s_qtok[tid] = tid >= R1 ? -1 : (g < RT - 1 ? p.row_tok[size_t(b) * p.r_max + g] : p.n_cur);
  }
  for (int i = tid; i < C; i += kRowsThreads) {         // the slot reserved for the current token is not written yet
    const int tok = map[i];
    s_tok[i] = tok == p.n_cur ? -1 : tok;
  }
  __syncthreads();

  // loads are numbered 0 .. 2 n_tiles - 1 (keys first, then values); load i uses stage i % kRowsStages
  auto issue = [&](int i) {
    const bool is_v = i >= n_tiles;
    const int t = is_v ? i - n_tiles : i;
    const int stage = i % kRowsStages;
    unsigned char* dst = ring + size_t(stage) * TILE_BYTES;
    mbar_expect_tx(&full[stage], uint32_t(TILE_BYTES));
#pragma unroll
    for (int hlf = 0; hlf < HALVES; ++hlf)
      rows_tma_load_2d(dst + hlf * (kRowsTile * 128), is_v ? &map_v : &map_k, hlf * 64, bh * C + t * kRowsTile, &full[stage]);
  };
  const int n_loads = 2 * n_tiles;
  if (tid == 0)
    for (int i = 0; i < min(kRowsStages, n_loads); ++i) issue(i);

  // ---- query block as A fragments: rows lane/4 and lane/4 + 8, columns 16 ks + (lane % 4) * 2 (+8) ----
  uint32_t qa[RB][KSTEPS][4];
#pragma unroll
  for (int k = 0; k < RB; ++k) {
    const T* qb = p.q + (size_t(bh) * RT + rb) * DH;
    const int r0 = k * kRowsMaxQ + (lane >> 2), r1 = r0 + 8, c0 = (lane & 3) * 2;
#pragma unroll
    for (int ks = 0; ks < KSTEPS; ++ks) {
      const int col = ks * 16 + c0;
      qa[k][ks][0] = r0 < R1 ? *reinterpret_cast<const uint32_t*>(qb + size_t(r0) * DH + col) : 0u;
      qa[k][ks][1] = r1 < R1 ? *reinterpret_cast<const uint32_t*>(qb + size_t(r1) * DH + col) : 0u;
      qa[k][ks][2] = r0 < R1 ? *reinterpret_cast<const uint32_t*>(qb + size_t(r0) * DH + col + 8) : 0u;
      qa[k][ks][3] = r1 < R1 ? *reinterpret_cast<const uint32_t*>(qb + size_t(r1) * DH + col + 8) : 0u;
    }
  }
  // the current token's own key: last row only (index C); every other row does not see it
  if (warp == kRowsWarps - 1) {
    const T* ql = p.q + (size_t(bh) * RT + (RT - 1)) * DH;
    const T* kn = p.k_new + size_t(bh) * DH;
    float dot = 0.f;
    if (has_last)
      for (int e = lane; e < DH; e += 32) dot = fmaf(__bfloat162float(ql[e]), __bfloat162float(kn[e]), dot);
    dot = warp_sum(dot);
    for (int r = lane; r < R1; r += 32) S[size_t(r) * SP + C] = (has_last && r == R1 - 1) ? dot * p.scale : -INFINITY;
  }

  bool failed = false;
  // ---- phase 1: logits, two tiles (two independent accumulator chains per warp) per block barrier ----
  int qt[RB][2];
#pragma unroll
  for (int k = 0; k < RB; ++k) { qt[k][0] = s_qtok[k * kRowsMaxQ + (lane >> 2)]; qt[k][1] = s_qtok[k * kRowsMaxQ + (lane >> 2) + 8]; }
  for (int t = 0; t < n_tiles; t += 2) {
    const int stage = t % kRowsStages;
    const uint32_t parity = uint32_t(t / kRowsStages) & 1u;
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2)
      if (!mbar_wait_bounded(&full[stage + h2], parity, failed ? kDrainPolls : kWaitPolls)) {
        if (!failed) set_error(p.err, ERRW_TIMEOUT);
        failed = true;
      }
    const uint32_t tile = smem_u32(ring + size_t(stage) * TILE_BYTES);
    float acc[RB][2][4];
#pragma unroll
    for (int k = 0; k < RB; ++k)
#pragma unroll
      for (int e = 0; e < 4; ++e) { acc[k][0][e] = 0.f; acc[k][1][e] = 0.f; }
    // ldmatrix.x4: matrix j holds keys warp*8 .. +7 (rows) x 8 columns starting at 8 * (4 q + j)
    const int krow = warp * 8 + (lane & 7), mj = lane >> 3;
#pragma unroll
    for (int q4 = 0; q4 < DH / 32; ++q4) {
      const int c16 = q4 * 4 + mj;                      // 16-byte chunk along dh (0 .. DH/8 - 1)
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2) {
        uint32_t bf[4];
        rows_ldmatrix_x4(tile + uint32_t(h2) * TILE_BYTES + uint32_t(c16 >> 3) * (kRowsTile * 128) + rows_swz(krow, c16 & 7), bf);
#pragma unroll
        for (int k = 0; k < RB; ++k) {                  // every row block uses the key fragments just read
          rows_mma(acc[k][h2], qa[k][2 * q4], bf[0], bf[1]);
          rows_mma(acc[k][h2], qa[k][2 * q4 + 1], bf[2], bf[3]);
        }
      }
    }
    // accumulator: rows lane/4 (+8), keys (lane % 4) * 2 (+1) of this warp's 8 in each tile
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      const int key0 = (t + h2) * kRowsTile + warp * 8 + (lane & 3) * 2;
#pragma unroll
      for (int k = 0; k < RB; ++k)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = k * kRowsMaxQ + (lane >> 2) + (e >> 1) * 8, key = key0 + (e & 1);
          if (r < R1 && key < C) {
            const int tok = s_tok[key];
            S[size_t(r) * SP + key] = (tok >= 0 && tok <= qt[k][e >> 1]) ? acc[k][h2][e] * p.scale : -INFINITY;
          }
        }
    }
    __syncthreads();                                    // everyone is done with these two stages
    if (tid == 0 && !failed) {
      if (t + kRowsStages < n_loads) issue(t + kRowsStages);
      if (t + kRowsStages + 1 < n_loads) issue(t + kRowsStages + 1);
    }
  }

  // ---- phase 2: per row, which logits are kept, softmax, weights (one warp per row) ----
  const int rows_n = C + 1;
  // The current token's row always needs a selection (it sees every slot) and goes first, to warp 0; the other rows
  // follow on warps 1..7, the ninth and later ones are stacked from warp 7 downwards, the next eight upwards again.
  for (int pass = 0; pass < 2 * RB; ++pass) {
    const int e = pass * kRowsWarps + ((pass & 1) ? kRowsWarps - 1 - warp : warp);   // entry 0: last row; entry e > 0: row e - 1
    if (e >= R1) continue;
    const int r = e == 0 ? R1 - 1 : e - 1;
    float* row = S + size_t(r) * SP;
    float* wout = p.weights ? p.weights + (size_t(bh) * RT + rb + r) * rows_n : nullptr;
    // this lane's logits as order-preserving keys, in registers (masked and out-of-range entries rank lowest)
    constexpr uint32_t kMasked = 0x007FFFFFu;           // key of -inf
    uint32_t kk[KPL];
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      const int i = j * 32 + lane;
      kk[j] = i < rows_n ? float_key(row[i]) : 0u;
    }
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < KPL; ++j) cnt += kk[j] > kMasked ? 1 : 0;
    cnt = __reduce_add_sync(0xffffffffu, cnt);
    uint32_t thr_key = 0u;
    if (cnt > p.topk) {
      // K-th largest key by bisection on the key's bits, most significant first: thr is the largest value with at
      // least K keys >= thr. A count is a compare and a ballot per 32 keys, all in registers: no atomics, no
      // shared-memory traffic, no dependence on how the logits are distributed. Bits above the highest bit in which
      // the candidates differ are taken as given.
      uint32_t kmin = 0xffffffffu, kmax = 0u;
#pragma unroll
      for (int j = 0; j < KPL; ++j)
        if (kk[j] > kMasked) { kmin = min(kmin, kk[j]); kmax = max(kmax, kk[j]); }
      kmin = __reduce_min_sync(0xffffffffu, kmin);
      kmax = __reduce_max_sync(0xffffffffu, kmax);
      const uint32_t diff = kmin ^ kmax;
      const int top = diff ? 31 - __clz(diff) : -1;
      uint32_t thr = top >= 31 ? 0u : (kmax & ~((2u << (top < 0 ? 0 : top)) - 1u));
      if (top < 0) thr = kmax;
      bool exact = false;
      for (int bit = top; bit >= 0; --bit) {
        const uint32_t cand = thr | (1u << bit);
        int c = 0;                                        // per-lane count, one warp-wide add per pass
#pragma unroll
        for (int j = 0; j < KPL; ++j) c += kk[j] >= cand ? 1 : 0;
        c = __reduce_add_sync(0xffffffffu, c);
        if (c >= p.topk) thr = cand;
        if (c == p.topk) { exact = true; break; }       // exactly K keys are >= thr: that is the kept set
      }
      thr_key = thr;
      int gt = 0, eq = 0;
      if (!exact) {
#pragma unroll
        for (int j = 0; j < KPL; ++j) { gt += kk[j] > thr ? 1 : 0; eq += kk[j] == thr ? 1 : 0; }
        gt = __reduce_add_sync(0xffffffffu, gt);
        eq = __reduce_add_sync(0xffffffffu, eq);
      }
      const int need = p.topk - gt;                     // how many of the keys equal to the threshold stay
      if (!exact && eq != need) {                       // equal logits at the threshold: the lowest indices stay
        if (lane == 0) {
          int left = need;
          for (int i = 0; i < rows_n; ++i)
            if (float_key(row[i]) == thr_key) { if (left > 0) --left; else row[i] = -INFINITY; }
        }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < KPL; ++j) {                 // (rare) the keys in registers follow the row
          const int i = j * 32 + lane;
          kk[j] = i < rows_n ? float_key(row[i]) : 0u;
        }
      }
    }
    // softmax over the kept logits, from the keys in registers (the key of a float is invertible): the largest key is
    // always kept, so it gives the maximum; weights go back to the row (phase 3 reads them) and out
    const uint32_t keep_from = thr_key > kMasked ? thr_key : kMasked + 1u;
    uint32_t kmax_all = 0u;
#pragma unroll
    for (int j = 0; j < KPL; ++j) kmax_all = max(kmax_all, kk[j]);
    kmax_all = __reduce_max_sync(0xffffffffu, kmax_all);
    const float mx = __uint_as_float((kmax_all & 0x80000000u) ? (kmax_all & 0x7fffffffu) : ~kmax_all);
    float part = 0.f;
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      const float l = __uint_as_float((kk[j] & 0x80000000u) ? (kk[j] & 0x7fffffffu) : ~kk[j]);
      const float e = kk[j] >= keep_from ? expf(l - mx) : 0.f;
      kk[j] = __float_as_uint(e);
      part += e;
    }
    part = warp_sum(part);
    const float inv = part > 0.f ? 1.f / part : 0.f;    // a padding row (nothing visible) keeps all-zero weights
#pragma unroll
    for (int j = 0; j < KPL; ++j) {
      const int i = j * 32 + lane;
      if (i < rows_n) {
        const float w = __uint_as_float(kk[j]) * inv;
        row[i] = w;
        if (wout) wout[i] = w;
      }
    }
  }
  __syncthreads();

  // ---- phase 3: O = P V. Warp w takes k-step w % 4 (16 keys) of every tile and column half w / 4, so the weight
  // fragments of a k-step are built by two warps instead of all eight; the partial outputs meet in shared memory ----
  constexpr int NTW = DH / 16;                          // 8-column n-tiles per warp (8 for dh 128, 4 for dh 64)
  const int my_ks = warp & 3, col_half = warp >> 2;
  float o[RB][NTW][4];
#pragma unroll
  for (int k = 0; k < RB; ++k)
#pragma unroll
    for (int j = 0; j < NTW; ++j) { o[k][j][0] = o[k][j][1] = o[k][j][2] = o[k][j][3] = 0.f; }
  for (int t = 0; t < n_tiles; t += 2) {
    const int li = n_tiles + t;
    const int stage = li % kRowsStages;
    const uint32_t parity = uint32_t(li / kRowsStages) & 1u;
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2)
      if (!mbar_wait_bounded(&full[stage + h2], parity, failed ? kDrainPolls : kWaitPolls)) {
        if (!failed) set_error(p.err, ERRW_TIMEOUT);
        failed = true;
      }
#pragma unroll
    for (int h2 = 0; h2 < 2; ++h2) {
      const uint32_t tile = smem_u32(ring + size_t(stage + h2) * TILE_BYTES);
      // A: weights of rows lane/4 (+8) for keys 16 my_ks + (lane % 4) * 2 (+1, +8, +9) of this tile, head + remainder
      const int key = (t + h2) * kRowsTile + my_ks * 16 + (lane & 3) * 2;
      uint32_t ah[RB][4], al[RB][4];
#pragma unroll
      for (int kb = 0; kb < RB; ++kb) {
        const int r0 = kb * kRowsMaxQ + (lane >> 2), r1 = r0 + 8;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int r = (e & 1) ? r1 : r0, k = key + (e >> 1) * 8;
          const float w0 = (r < R1 && k < C) ? S[size_t(r) * SP + k] : 0.f;
          const float w1 = (r < R1 && k + 1 < C) ? S[size_t(r) * SP + k + 1] : 0.f;
          const __nv_bfloat16 h0 = __float2bfloat16_rn(w0), h1 = __float2bfloat16_rn(w1);
          ah[kb][e] = rows_pack_bf16(__bfloat162float(h0), __bfloat162float(h1));
          al[kb][e] = rows_pack_bf16(w0 - __bfloat162float(h0), w1 - __bfloat162float(h1));
        }
      }
      // B (transposed load): matrix j: keys 16 my_ks + 8 (j % 2) .. +7 (rows of the tile) x the columns of n-tile j / 2
      const int vrow = my_ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
      for (int nt = 0; nt < NTW; nt += 2) {
        const int c16 = col_half * NTW + nt + (lane >> 4);
        uint32_t bf[4];
        rows_ldmatrix_x4_trans(tile + uint32_t(c16 >> 3) * (kRowsTile * 128) + rows_swz(vrow, c16 & 7), bf);
#pragma unroll
        for (int kb = 0; kb < RB; ++kb) {               // every row block uses the value fragments just read
          rows_mma(o[kb][nt], ah[kb], bf[0], bf[1]);
          rows_mma(o[kb][nt], al[kb], bf[0], bf[1]);
          rows_mma(o[kb][nt + 1], ah[kb], bf[2], bf[3]);
          rows_mma(o[kb][nt + 1], al[kb], bf[2], bf[3]);
        }
      }
    }
    __syncthreads();
    if (tid == 0 && !failed) {
      if (li + kRowsStages < n_loads) issue(li + kRowsStages);
      if (li + kRowsStages + 1 < n_loads) issue(li + kRowsStages + 1);
    }
  }

  // ---- the four k-step warps of a column half add up through shared memory (the ring is free now), one row block
  // after the other, then rows < R1 go out; the last row also gets the current token's own value row ----
  {
    float* part = reinterpret_cast<float*>(ring);       // [4 k-steps][16 rows][DH] floats: at most 32 KB
    const T* vn = p.v_new + size_t(bh) * DH;
    const float w_own = has_last ? S[size_t(R1 - 1) * SP + C] : 0.f;
#pragma unroll
    for (int kb = 0; kb < RB; ++kb) {
      if (kb * kRowsMaxQ >= R1) break;                  // (the same in every thread)
      if (kb > 0) __syncthreads();                      // the previous block's sums have been read
#pragma unroll
      for (int nt = 0; nt < NTW; ++nt) {
        const int col = col_half * (DH / 2) + nt * 8 + (lane & 3) * 2;
#pragma unroll
        for (int hrow = 0; hrow < 2; ++hrow) {
          const int r = (lane >> 2) + hrow * 8;
          float* d = part + (size_t(my_ks) * 16 + r) * DH + col;
          d[0] = o[kb][nt][hrow * 2];
          d[1] = o[kb][nt][hrow * 2 + 1];
        }
      }
      __syncthreads();
      const int rows_here = min(kRowsMaxQ, R1 - kb * kRowsMaxQ);
      for (int i = tid; i < rows_here * (DH / 2); i += kRowsThreads) {
        const int rl = i / (DH / 2), col = (i % (DH / 2)) * 2, r = kb * kRowsMaxQ + rl;
        float a0 = 0.f, a1 = 0.f;
#pragma unroll
        for (int q4 = 0; q4 < 4; ++q4) {
          const float* d = part + (size_t(q4) * 16 + rl) * DH + col;
          a0 += d[0];
          a1 += d[1];
        }
        if (has_last && r == R1 - 1) {
          a0 = fmaf(w_own, __bfloat162float(vn[col]), a0);
          a1 = fmaf(w_own, __bfloat162float(vn[col + 1]), a1);
        }
        *reinterpret_cast<uint32_t*>(p.out + (size_t(bh) * RT + rb + r) * DH + col) = rows_pack_bf16(a0, a1);
      }
    }
  }
  // ---- admit: the current token's rows go into their slot (all tiles of this pair have been consumed) ----
  if (p.admit_slot != nullptr) {
    const int s = p.admit_slot[b];
    if (s >= 0 && s < C) {
      constexpr int V16 = DH * 2 / 16;
      unsigned char* kd = reinterpret_cast<unsigned char*>(p.Kc) + (size_t(bh) * C + s) * DH * 2;
      unsigned char* vd = reinterpret_cast<unsigned char*>(p.Vc) + (size_t(bh) * C + s) * DH * 2;
      const unsigned char* knew = reinterpret_cast<const unsigned char*>(p.k_new) + size_t(bh) * DH * 2;
      const unsigned char* vnew = reinterpret_cast<const unsigned char*>(p.v_new) + size_t(bh) * DH * 2;
      if (tid < V16) reinterpret_cast<uint4*>(kd)[tid] = reinterpret_cast<const uint4*>(knew)[tid];
      else if (tid < 2 * V16) reinterpret_cast<uint4*>(vd)[tid - V16] = reinterpret_cast<const uint4*>(vnew)[tid - V16];
    } else if (tid == 0) {
      set_error(p.err, ERRW_BOUNDS);
    }
  }
}

}  // namespace adore
