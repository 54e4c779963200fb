// Release / admit / rebuild-list selection and the slot map (one CTA per sequence).
//
// Section 2.2: when the cache is full the retained token with the lowest controller score is
// released and the newest token is appended; one decision per token serves all layers and heads.
// Section 2.3: among released tokens, the R with the highest score are rebuilt for the next step.
// Tokens are compared by (score, position): higher score first, the newer token on equal scores.
// The order is materialised as one 64-bit key per token and sorted in shared memory.
#pragma once

#include <limits.h>

#include "common.cuh"

namespace adore {

// ---- block-wide helpers (any blockDim.x that is a multiple of 32, scratch of 64 words) --------
__device__ __forceinline__ int block_sum_i(int v, int* tmp) {
  v = warp_sum(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = 0;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) r += tmp[w];
  return r;
}
__device__ __forceinline__ int block_min_i(int v, int* tmp) {
  v = warp_min(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = v;
  __syncthreads();
  int r = INT_MAX;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) r = min(r, tmp[w]);
  return r;
}
__device__ __forceinline__ unsigned long long block_min_u64(unsigned long long v, unsigned long long* tmp) {
  v = warp_min(v);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long r = ~0ull;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) r = tmp[w] < r ? tmp[w] : r;
  return r;
}
// Largest 64-bit value of a warp: the high words first, then the low words of the lanes that hold the largest high word.
__device__ __forceinline__ unsigned long long warp_max_u64(unsigned long long v) {
  const uint32_t hi = uint32_t(v >> 32);
  const uint32_t hmax = __reduce_max_sync(0xffffffffu, hi);
  const uint32_t lmax = __reduce_max_sync(0xffffffffu, hi == hmax ? uint32_t(v) : 0u);
  return (static_cast<unsigned long long>(hmax) << 32) | lmax;
}
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v, unsigned long long* tmp) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const unsigned long long t = __shfl_xor_sync(0xffffffffu, v, o);
    v = t > v ? t : v;
  }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) tmp[threadIdx.x >> 5] = v;
  __syncthreads();
  unsigned long long r = 0ull;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) r = tmp[w] > r ? tmp[w] : r;
  return r;
}
// Exclusive position of this thread's flag among the block's flags (thread order); total out.
__device__ __forceinline__ int block_rank(bool flag, int* tmp, int* total) {
  const unsigned bal = __ballot_sync(0xffffffffu, flag);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) tmp[warp] = __popc(bal);
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) { const int c = tmp[w]; if (w < warp) base += c; tot += c; }
  *total = tot;
  return base + __popc(bal & ((1u << lane) - 1u));
}

// Exclusive prefix sum of v over the block's threads (thread order); total out. tmp: 64 words.
__device__ __forceinline__ int block_scan_excl(int v, int* tmp, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int t = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += t;
  }
  __syncthreads();
  if (lane == 31) tmp[warp] = incl;
  __syncthreads();
  int base = 0, tot = 0;
  for (int w = 0; w < int(blockDim.x >> 5); ++w) { const int c = tmp[w]; if (w < warp) base += c; tot += c; }
  *total = tot;
  return base + incl - v;
}

// ---- bitonic sort, DESCENDING, P a power of two -------------------------------------------------
// Each warp owns a contiguous block of E = 32*R keys and keeps them in registers (R per lane, key
// x = base + 32*r + lane). Compare-exchange stages whose partners are less than E apart never leave
// the warp: a distance below 32 is a shuffle, a distance of 32 or more is another register of the same
// lane. Only the stages that cross warps go through shared memory, one block barrier each.
template <int R>
__device__ __forceinline__ void bitonic_warp_run(unsigned long long (&v)[R], int base, int lane, int k, int j_start) {
#pragma unroll
  for (int sft = 9; sft >= 0; --sft) {               // j = 512 .. 1, compile-time after unrolling
    const int j = 1 << sft;
    if (j >= 32 * R || j > j_start) continue;
    if (j >= 32) {
      const int dr = j >> 5;
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if ((r & dr) == 0) {
          const bool desc = ((base + r * 32 + lane) & k) == 0;
          const unsigned long long a = v[r], c = v[r | dr];
          if (desc ? (a < c) : (a > c)) { v[r] = c; v[r | dr] = a; }
        }
      }
    } else {
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const unsigned long long other = __shfl_xor_sync(0xffffffffu, v[r], j);
        const bool desc = ((base + r * 32 + lane) & k) == 0;
        const bool take_max = ((lane & j) == 0) == desc;
        const unsigned long long hi = v[r] > other ? v[r] : other, lo = v[r] > other ? other : v[r];
        v[r] = take_max ? hi : lo;
      }
    }
  }
}

template <int R>
__device__ __forceinline__ void bitonic_sort_desc_regs(unsigned long long* keys, int P) {
  constexpr int E = 32 * R;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const bool active = warp < P / E;
  const int base = warp * E;
  unsigned long long v[R];
  __syncthreads();                                    // the keys were written by arbitrary threads
#pragma unroll
  for (int r = 0; r < R; ++r) v[r] = active ? keys[base + r * 32 + lane] : 0ull;
  for (int k = 2; k <= E; k <<= 1) bitonic_warp_run<R>(v, base, lane, k, k >> 1);
  for (int k = 2 * E; k <= P; k <<= 1) {
    if (active) {
#pragma unroll
      for (int r = 0; r < R; ++r) keys[base + r * 32 + lane] = v[r];
    }
    __syncthreads();
    for (int j = k >> 1; j >= E; j >>= 1) {           // partners in other warps' blocks
      for (int t = threadIdx.x; t < (P >> 1); t += blockDim.x) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int l = i | j;
        const unsigned long long a = keys[i], c = keys[l];
        const bool desc = (i & k) == 0;
        if (desc ? (a < c) : (a > c)) { keys[i] = c; keys[l] = a; }
      }
      __syncthreads();
    }
#pragma unroll
    for (int r = 0; r < R; ++r) v[r] = active ? keys[base + r * 32 + lane] : 0ull;
    bitonic_warp_run<R>(v, base, lane, k, E >> 1);
  }
  if (active) {
#pragma unroll
    for (int r = 0; r < R; ++r) keys[base + r * 32 + lane] = v[r];
  }
  __syncthreads();
}

// Small inputs (P < 64): everything in shared memory.
__device__ inline void bitonic_sort_desc_small(unsigned long long* keys, int P) {
  for (int k = 2; k <= P; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      __syncthreads();
      for (int t = threadIdx.x; t < (P >> 1); t += blockDim.x) {
        const int i = ((t & ~(j - 1)) << 1) | (t & (j - 1));
        const int l = i | j;
        const unsigned long long a = keys[i], c = keys[l];
        const bool desc = (i & k) == 0;
        if (desc ? (a < c) : (a > c)) { keys[i] = c; keys[l] = a; }
      }
    }
  }
  __syncthreads();
}

// All threads of the block call it; blockDim.x a multiple of 32; P <= 512 * (blockDim.x / 32).
__device__ inline void bitonic_sort_desc(unsigned long long* keys, int P) {
  const int nw = blockDim.x >> 5;
  if (P < 64) { bitonic_sort_desc_small(keys, P); return; }
  const int E = max(64, P / nw);                      // keys per warp
  if (E == 64) bitonic_sort_desc_regs<2>(keys, P);
  else if (E == 128) bitonic_sort_desc_regs<4>(keys, P);
  else if (E == 256) bitonic_sort_desc_regs<8>(keys, P);
  else bitonic_sort_desc_regs<16>(keys, P);
}

struct SelectParams {
  int B, C, m, r_max, n;      // n: position of the token being admitted
  int max_tokens;
  int explicit_mode;
  int P;                      // sort width: power of two >= number of candidate entries
  const int* slot_tok_old;    // [B,C]
  const uint8_t* slot_role_old;
  int* slot_tok_new;
  uint8_t* slot_role_new;
  int* tok_slot;              // [B,max_tokens]
  const float* score;         // [B,max_tokens]
  const int* explicit_list;   // [B,r_in]
  const int* explicit_count;  // [B]
  int r_in;
  int* admit_slot;            // [B]
  int* evicted_tok;           // [B]
  int* rebuild_tok;           // [B,r_max]
  int* rebuild_slot;          // [B,r_max]
  int* rebuild_count;         // [B]
  unsigned* err;
  // decode step: the CTA that finishes last also compacts all sequences' lists into the row table of the rebuild
  int* row_b;                 // [B * r_max] or null (no table: the bulk load builds it with row_table_kernel)
  int* row_tok;
  int* row_slot;
  int* row_total;
  unsigned long long* rows_accum;   // running total of rebuilt rows, or null
  unsigned* done_count;       // arrivals of this launch's CTAs; left at zero by the last one
};

__host__ __device__ inline size_t select_smem_bytes(int C, int P) {
  // keys[P] u64 | tok[C] | lst[C] | slots[C] int | 64 words scratch + 512 offsets (row table) | role[C] u8 (padded) | 32 u64
  return sizeof(unsigned long long) * size_t(P) + sizeof(int) * 3 * size_t(C) + ((size_t(C) + 15) & ~size_t(15)) +
         sizeof(int) * (64 + 512) + sizeof(unsigned long long) * 32;
}

struct SelectSmem {
  unsigned long long* keys;
  int* tok;
  int* lst;
  int* slots;
  uint8_t* role;
  int* tmp;
  unsigned long long* tmp64;
  __device__ SelectSmem(unsigned char* base, int C, int P) {
    tmp64 = reinterpret_cast<unsigned long long*>(base);
    keys = tmp64 + 32;
    tok = reinterpret_cast<int*>(keys + P);
    lst = tok + C;
    slots = lst + C;
    tmp = slots + C;
    role = reinterpret_cast<uint8_t*>(tmp + 64 + 512);     // (selection kernels run with at most 512 threads)
  }
};

constexpr int kSelectIterMax = 16;     // lists up to this length are picked by repeated block-wide maxima
constexpr int kSelectIterKeys = 16;    // keys a thread holds for that (512 threads x 16 = the largest token table)

__device__ inline int place_rebuild_list(const struct SelectParams& p, const struct SelectSmem& sm, int b, int* tok_slot, int found);

// Candidate keys -> sorted -> first r_max distinct tokens -> ascending empty slots.
// Expects sm.tok / sm.role to hold the map with the new token already placed. Returns the count.
__device__ inline int assign_rebuild_list(const SelectParams& p, const SelectSmem& sm, int b, int* tok_slot,
                                          int n_seen) {
  const int tid = threadIdx.x, NT = blockDim.x;
  const float* score = p.score + size_t(b) * p.max_tokens;
  if (p.explicit_mode) {
    const int cnt = p.explicit_list ? min(p.explicit_count[b], p.r_in) : 0;
    for (int i = tid; i < p.P; i += NT) {
      unsigned long long key = 0ull;
      if (i < cnt) {
        const int e = p.explicit_list[size_t(b) * p.r_in + i];
        if (e < 0 || e >= n_seen) set_error(p.err, ERRW_BAD_LIST);
        else if (tok_slot[e] < 0) key = value_key(score[e], e);
      }
      sm.keys[i] = key;
    }
  } else if (p.r_max <= kSelectIterMax && p.P <= kSelectIterKeys * NT) {
    // A short list out of many released tokens (the paper's R = 8 of thousands): no sort. Every thread keeps its
    // candidates' keys in registers and the block takes the largest key below the previous one, r_max times (keys are
    // distinct: the token position is part of the key).
    unsigned long long k[kSelectIterKeys];
#pragma unroll
    for (int j = 0; j < kSelectIterKeys; ++j) {
      const int i = tid + j * NT;
      k[j] = (i < n_seen && tok_slot[i] < 0) ? value_key(score[i], i) : 0ull;
    }
    int found = 0;
    const int NW = NT >> 5, lane = tid & 31, warp = tid >> 5;
    if (p.P >= NW * p.r_max) {
      // Two levels, two block barriers: every warp picks the r_max largest of its own keys (a warp-wide maximum of a
      // 64-bit key = two 32-bit ones: the score part, then the position among the lanes that hold that score), the
      // candidates of all warps meet in shared memory (the key array is free here) and warp 0 picks among them.
      unsigned long long prev = ~0ull;
      for (int r = 0; r < p.r_max; ++r) {
        unsigned long long m = 0ull;
#pragma unroll
        for (int j = 0; j < kSelectIterKeys; ++j) m = (k[j] < prev && k[j] > m) ? k[j] : m;
        m = warp_max_u64(m);
        if (lane == 0) sm.keys[warp * p.r_max + r] = m;    // (0 once the warp has run out of released tokens)
        prev = m == 0ull ? 0ull : m;
      }
      __syncthreads();
      if (warp == 0) {
        unsigned long long c[kSelectIterKeys / 2];           // 16 warps x 16 candidates at most = 8 per lane
#pragma unroll
        for (int j = 0; j < kSelectIterKeys / 2; ++j) {
          const int i = lane + 32 * j;
          c[j] = i < NW * p.r_max ? sm.keys[i] : 0ull;
        }
        unsigned long long top = ~0ull;
        for (int r = 0; r < p.r_max; ++r) {
          unsigned long long m = 0ull;
#pragma unroll
          for (int j = 0; j < kSelectIterKeys / 2; ++j) m = (c[j] < top && c[j] > m) ? c[j] : m;
          m = warp_max_u64(m);
          if (m == 0ull) break;
          if (lane == 0) sm.lst[r] = int(m & 0xffffffffull);
          top = m;
          ++found;
        }
        if (lane == 0) sm.tmp[0] = found;
      }
      __syncthreads();
      found = sm.tmp[0];
      return place_rebuild_list(p, sm, b, tok_slot, found);
    }
    unsigned long long prev = ~0ull;
    for (int r = 0; r < p.r_max; ++r) {
      unsigned long long m = 0ull;
#pragma unroll
      for (int j = 0; j < kSelectIterKeys; ++j) m = (k[j] < prev && k[j] > m) ? k[j] : m;
      m = block_max_u64(m, sm.tmp64);
      if (m == 0ull) break;                                 // block-uniform: no released token is left
      if (tid == 0) sm.lst[r] = int(m & 0xffffffffull);
      prev = m;
      ++found;
    }
    return place_rebuild_list(p, sm, b, tok_slot, found);
  } else {
    for (int i = tid; i < p.P; i += NT)
      sm.keys[i] = (i < n_seen && tok_slot[i] < 0) ? value_key(score[i], i) : 0ull;
  }
  bitonic_sort_desc(sm.keys, p.P);
  int found = 0;
  for (int i0 = 0; i0 < p.P && found < p.r_max; i0 += NT) {
    if (sm.keys[i0] == 0ull) break;                       // sorted: nothing but padding follows
    const int i = i0 + tid;
    const bool f = i < p.P && sm.keys[i] != 0ull && (i == 0 || sm.keys[i] != sm.keys[i - 1]);
    int tot;
    const int pos = found + block_rank(f, sm.tmp, &tot);
    if (f && pos < p.r_max) sm.lst[pos] = int(sm.keys[i] & 0xffffffffull);
    found += tot;
  }
  return place_rebuild_list(p, sm, b, tok_slot, found);
}

// The first min(found, r_max) tokens of sm.lst (most valuable first) take the empty slots in ascending order.
__device__ inline int place_rebuild_list(const SelectParams& p, const SelectSmem& sm, int b, int* tok_slot, int found) {
  const int tid = threadIdx.x, NT = blockDim.x;
  const int cnt = min(found, p.r_max);
  int seen = 0;
  __syncthreads();
  for (int s0 = 0; s0 < p.C && seen < cnt; s0 += NT) {
    const int s = s0 + tid;
    const bool f = s < p.C && sm.role[s] == ROLE_EMPTY;
    int tot;
    const int pos = seen + block_rank(f, sm.tmp, &tot);
    if (f && pos < cnt) sm.slots[pos] = s;
    seen += tot;
  }
  __syncthreads();
  for (int j = tid; j < p.r_max; j += NT) {
    int tok = -1, s = -1;
    if (j < cnt) {
      tok = sm.lst[j];
      s = sm.slots[j];
      sm.tok[s] = tok;
      sm.role[s] = ROLE_REBUILT;
      tok_slot[tok] = s;
    }
    p.rebuild_tok[size_t(b) * p.r_max + j] = tok;
    p.rebuild_slot[size_t(b) * p.r_max + j] = s;
  }
  if (tid == 0) p.rebuild_count[b] = cnt;
  __syncthreads();
  return cnt;
}

// Turns the per-sequence rebuild lists into one compact row table (b-major, list order): CTA b sums
// the counts of the sequences before it and writes its own rows. One small launch after the selection.
__global__ void __launch_bounds__(128) row_table_kernel(const int* rebuild_tok, const int* rebuild_slot,
                                                        const int* rebuild_count, int B, int r_max, int* row_b, int* row_tok,
                                                        int* row_slot, int* row_total, unsigned long long* rows_accum) {
  __shared__ int tmp[64];
  const int b = blockIdx.x, tid = threadIdx.x;
  let_next_grid_start();
  wait_for_prior_grid();
  int before = 0, all = 0;
  for (int i = tid; i < B; i += blockDim.x) {
    const int c = rebuild_count[i];
    all += c;
    if (i < b) before += c;
  }
  const int off = block_sum_i(before, tmp);
  const int total = block_sum_i(all, tmp);
  const int cnt = rebuild_count[b];
  for (int j = tid; j < cnt; j += blockDim.x) {
    row_b[off + j] = b;
    row_tok[off + j] = rebuild_tok[size_t(b) * r_max + j];
    row_slot[off + j] = rebuild_slot[size_t(b) * r_max + j];
  }
  if (b == 0 && tid == 0) {
    *row_total = total;
    if (rows_accum) *rows_accum += static_cast<unsigned long long>(total);
  }
}

// Called by every thread of every CTA of a decode step's selection launch once its sequence's list is written: the CTA
// that arrives last turns the per-sequence lists into the compact row table (b-major, list order) that the gather and
// the GEMM of the rebuild walk, so that no further launch stands between the selection and them.
__device__ inline void select_finish_row_table(const SelectParams& p, int* s_tmp) {
  if (p.row_b == nullptr) return;
  const int tid = threadIdx.x, NT = blockDim.x;
  __threadfence();                                   // this CTA's list is visible before its arrival is
  __syncthreads();
  if (tid == 0) s_tmp[63] = (atomicAdd(p.done_count, 1u) == unsigned(p.B - 1)) ? 1 : 0;
  __syncthreads();
  if (s_tmp[63] == 0) return;
  __threadfence();
  // offsets: sequences in chunks of blockDim.x, an exclusive scan of the counts per chunk (every thread ends up with the
  // same running total); then all threads copy the chunk's entries, one (sequence, list position) pair each per round
  int* s_off = s_tmp + 64;                           // [blockDim.x], provided by the caller behind its scratch words
  int base = 0;
  for (int b0 = 0; b0 < p.B; b0 += NT) {
    const int b = b0 + tid;
    const int mine = b < p.B ? min(__ldcg(p.rebuild_count + b), p.r_max) : 0;
    int tot;
    const int excl = block_scan_excl(mine, s_tmp, &tot);
    s_off[tid] = base + excl;
    __syncthreads();
    const int nb = min(NT, p.B - b0);
#pragma unroll 4
    for (int idx = tid; idx < nb * p.r_max; idx += NT) {
      const int bb = idx / p.r_max, j = idx - bb * p.r_max;
      const int next = bb + 1 < nb ? s_off[bb + 1] : base + tot;
      if (j < next - s_off[bb]) {
        const size_t src = size_t(b0 + bb) * p.r_max + j;
        p.row_b[s_off[bb] + j] = b0 + bb;
        p.row_tok[s_off[bb] + j] = __ldcg(p.rebuild_tok + src);
        p.row_slot[s_off[bb] + j] = __ldcg(p.rebuild_slot + src);
      }
    }
    base += tot;
    __syncthreads();
  }
  if (tid == 0) {
    *p.row_total = base;
    if (p.rows_accum) *p.rows_accum += static_cast<unsigned long long>(base);
    *p.done_count = 0u;                              // ready for the next launch
  }
}

// One decode step's selection for sequence blockIdx.x.
__device__ inline void select_step(const SelectParams& p, unsigned char* smem) {
  const int b = blockIdx.x, tid = threadIdx.x, NT = blockDim.x, C = p.C;
  SelectSmem sm(smem, C, p.P);
  int* tok_slot = p.tok_slot + size_t(b) * p.max_tokens;
  const float* score = p.score + size_t(b) * p.max_tokens;
  // 1. rebuilt states live for one step: free them
  for (int s = tid; s < C; s += NT) {
    int t = p.slot_tok_old[size_t(b) * C + s];
    uint8_t r = p.slot_role_old[size_t(b) * C + s];
    if (r == ROLE_REBUILT) { tok_slot[t] = -1; t = -1; r = ROLE_EMPTY; }
    sm.tok[s] = t;
    sm.role[s] = r;
  }
  __syncthreads();
  // 2. + 3. One pass over the map and ONE block-wide reduction give the number of retained tokens, the least valuable of
  // them and the lowest empty slot. A full cache releases that token; the new token takes the lowest empty slot, which
  // is the released token's own if that lies lower.
  int cnt = 0, emin = INT_MAX;
  unsigned long long kmin = ~0ull;
  for (int s = tid; s < C; s += NT) {
    const uint8_t r = sm.role[s];
    if (r == ROLE_RETAINED) {
      ++cnt;
      const unsigned long long k = value_key(score[sm.tok[s]], sm.tok[s]);
      kmin = k < kmin ? k : kmin;
    } else if (r == ROLE_EMPTY) {
      emin = min(emin, s);
    }
  }
  cnt = warp_sum(cnt);
  kmin = warp_min(kmin);
  emin = warp_min(emin);
  if ((tid & 31) == 0) { sm.tmp[tid >> 5] = cnt; sm.tmp[32 + (tid >> 5)] = emin; sm.tmp64[tid >> 5] = kmin; }
  if (tid == 0) sm.tmp[31] = INT_MAX;                     // the released token's slot, written below by the thread that holds it
  __syncthreads();
  int n_ret = 0;
  emin = INT_MAX;
  kmin = ~0ull;
  for (int w = 0; w < (NT >> 5); ++w) {
    n_ret += sm.tmp[w];
    emin = min(emin, sm.tmp[32 + w]);
    kmin = sm.tmp64[w] < kmin ? sm.tmp64[w] : kmin;
  }
  const int evicted = (n_ret >= p.m) ? int(kmin & 0xffffffffull) : -1;
  if (evicted >= 0)
    for (int s = tid; s < C; s += NT)
      if (sm.tok[s] == evicted) { sm.tok[s] = -1; sm.role[s] = ROLE_EMPTY; tok_slot[evicted] = -1; sm.tmp[31] = s; }
  __syncthreads();
  if (tid == 0) {
    const int amin = min(emin, sm.tmp[31]);
    if (amin < C) { sm.tok[amin] = p.n; sm.role[amin] = ROLE_RETAINED; tok_slot[p.n] = amin; }
    else set_error(p.err, ERRW_BOUNDS);
    p.admit_slot[b] = amin < C ? amin : -1;
    p.evicted_tok[b] = evicted;
  }
  __syncthreads();
  // 4./5. rebuild list among the released tokens, into the empty slots
  assign_rebuild_list(p, sm, b, tok_slot, p.n);
  for (int s = tid; s < C; s += NT) {
    p.slot_tok_new[size_t(b) * C + s] = sm.tok[s];
    p.slot_role_new[size_t(b) * C + s] = sm.role[s];
  }
  select_finish_row_table(p, sm.tmp);
}

// Bulk load of T tokens into an empty cache: the newest token plus the min(m-1, T-1) most
// valuable earlier ones are retained, in ascending position from slot 0; then the rebuild list.
// p.n = T (tokens seen), p.P >= T.
__device__ inline void select_bulk(const SelectParams& p, unsigned char* smem) {
  const int b = blockIdx.x, tid = threadIdx.x, NT = blockDim.x, C = p.C, T = p.n;
  SelectSmem sm(smem, C, p.P);
  int* tok_slot = p.tok_slot + size_t(b) * p.max_tokens;
  const float* score = p.score + size_t(b) * p.max_tokens;
  for (int s = tid; s < C; s += NT) { sm.tok[s] = -1; sm.role[s] = ROLE_EMPTY; }
  for (int i = tid; i < p.P; i += NT) sm.keys[i] = (i < T - 1) ? value_key(score[i], i) : 0ull;
  for (int i = tid; i < T; i += NT) tok_slot[i] = -1;
  bitonic_sort_desc(sm.keys, p.P);
  const int n_keep = min(p.m - 1, T - 1);
  for (int i = tid; i < n_keep; i += NT) tok_slot[int(sm.keys[i] & 0xffffffffull)] = -2;   // mark
  if (tid == 0) tok_slot[T - 1] = -2;
  __syncthreads();
  int placed = 0;
  for (int t0 = 0; t0 < T; t0 += NT) {
    const int t = t0 + tid;
    const bool f = t < T && tok_slot[t] == -2;
    int tot;
    const int pos = placed + block_rank(f, sm.tmp, &tot);
    if (f) { sm.tok[pos] = t; sm.role[pos] = ROLE_RETAINED; tok_slot[t] = pos; }
    placed += tot;
  }
  if (tid == 0) { p.admit_slot[b] = -1; p.evicted_tok[b] = -1; }
  __syncthreads();
  if (p.explicit_mode) {     // no candidates are named for a prompt
    for (int j = tid; j < p.r_max; j += NT) { p.rebuild_tok[size_t(b) * p.r_max + j] = -1; p.rebuild_slot[size_t(b) * p.r_max + j] = -1; }
    if (tid == 0) p.rebuild_count[b] = 0;
    __syncthreads();
  } else {
    assign_rebuild_list(p, sm, b, tok_slot, T);
  }
  for (int s = tid; s < C; s += NT) {
    p.slot_tok_new[size_t(b) * C + s] = sm.tok[s];
    p.slot_role_new[size_t(b) * C + s] = sm.role[s];
  }
}

// Row table of every occupied slot (for filling a layer): one CTA.
__global__ void resident_rows_kernel(const int* slot_tok, int B, int C, int* row_b, int* row_tok, int* row_slot,
                                     int* row_total) {
  __shared__ int tmp[64];
  int base = 0;
  for (int i0 = 0; i0 < B * C; i0 += blockDim.x) {
    const int i = i0 + threadIdx.x;
    const bool f = i < B * C && slot_tok[i] >= 0;
    int tot;
    const int pos = base + block_rank(f, tmp, &tot);
    if (f) { row_b[pos] = i / C; row_tok[pos] = slot_tok[i]; row_slot[pos] = i % C; }
    base += tot;
  }
  if (threadIdx.x == 0) *row_total = base;
}

}  // namespace adore
