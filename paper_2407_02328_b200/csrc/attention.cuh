// Decode attention over the slot cache with top-K masking and weight emission.
//
// Computes, per (sequence b, head h), the target attention of Section 2.1 (unnumbered equation
// after Eq. 1) / Section 2.3: logits of the query against every occupied slot and against the
// current token's own key, only the K largest logits keep a weight (Section 2.2, first bullet),
// softmax over the kept ones, weighted sum of the kept value rows. The kept weights are written
// out per slot. Finally the current token's key/value row is written into its slot (append of
// the most recent state, Section 2.2 third bullet).
//
// This header holds the phases the attention kernels share: given the logits of a (b, h) pair in shared
// memory, phase 2 finds the K-th largest logit with a 4-pass radix select, phase 3 is the softmax, phase 4
// reads ONLY the kept value rows, and the tail writes the output and the current token's row. Phase 1 (the
// logits) belongs to the kernels: attention_tma.cuh stages the contiguous C*dh key block of a pair through
// shared memory, attention_split.cuh spreads it over a thread-block cluster.
#pragma once

#include "common.cuh"

namespace adore {

template <typename T>
struct AttnParams {
  const T* q;            // [B,H,DH]
  const T* k_new;        // [B,H,DH]
  const T* v_new;        // [B,H,DH]
  T* out;                // [B,H,DH]
  float* weights;        // [B,H,C+1] or nullptr
  T* Kc;                 // layer base [B,H,C,DH]
  T* Vc;
  const int* slot_tok;   // [B,C] map the cache rows currently follow (<0: empty)
  const int* admit_slot; // [B] slot that receives the new row, or nullptr
  int B, H, C, topk;
  float scale;           // 1/sqrt(DH)
  unsigned* err;
  // Several query rows per (b, h) (Section 2.3: the rebuilt tokens' rows and the current token's; 1 = the plain
  // decode step). q, out and weights then hold rows_q rows per pair, item = (b*H + h) * rows_q + i. Row i < rows_q-1
  // belongs to token row_tok[b*r_max + i] (< 0: padding, the row's output is zero), the last row to token n_cur. A row
  // sees the slots whose token position is at most its own, never the slot reserved for n_cur (not written yet), and
  // the current token's own row (index C) only if it is the last row.
  int rows_q;
  const int* row_tok;    // [B, r_max] or nullptr
  int r_max, n_cur;
  // A launch of the tensor-core rows kernel may cover a group of a pair's rows only: rows row_base .. row_base +
  // rows_q - 1 of rows_total (0: the launch covers all rows_q rows). q, out and weights keep rows_total rows per pair.
  int row_base, rows_total;
};

constexpr int kAttnThreads = 256;
constexpr int kAttnUnroll = 4;

__host__ __device__ inline size_t attn_smem_bytes(int C, int DH, int threads = kAttnThreads) {
  const int cp = (C + 1 + 3) & ~3;
  return sizeof(float) * cp + sizeof(int) * cp + sizeof(unsigned) * 256 +
         sizeof(float) * (threads / 32) * DH + sizeof(float) * 64;
}

// Who "the block" of the shared phases is: the whole CTA, or one 128-thread group of a CTA that works on two pairs at
// once (threads 0..127 and 128..255, each group with a named barrier of its own; further warps of the CTA stay out).
struct CtaScope {
  static __device__ __forceinline__ int tid() { return threadIdx.x; }
  static __device__ __forceinline__ void sync() { __syncthreads(); }
};
struct GroupScope {
  static __device__ __forceinline__ int tid() { return threadIdx.x & 127; }
  static __device__ __forceinline__ void sync() { asm volatile("bar.sync %0, 128;" ::"r"(1 + (threadIdx.x >> 7)) : "memory"); }
};

template <int NT, typename SY = CtaScope>
__device__ __forceinline__ float block_sum_f(float v, float* tmp) {
  const int lane = SY::tid() & 31, warp = SY::tid() >> 5;
  v = warp_sum(v);
  SY::sync();                       // tmp may still be read from a previous reduction
  if (lane == 0) tmp[warp] = v;
  SY::sync();
  float r = 0.f;
#pragma unroll
  for (int w = 0; w < NT / 32; ++w) r += tmp[w];
  return r;
}
template <int NT, typename SY = CtaScope>
__device__ __forceinline__ float block_max_f(float v, float* tmp) {
  const int lane = SY::tid() & 31, warp = SY::tid() >> 5;
  v = warp_max(v);
  SY::sync();
  if (lane == 0) tmp[warp] = v;
  SY::sync();
  float r = tmp[0];
#pragma unroll
  for (int w = 1; w < NT / 32; ++w) r = fmaxf(r, tmp[w]);
  return r;
}

// Shared-memory carve-up common to the attention kernels.
template <int DH, int NT = kAttnThreads>
struct AttnSmem {
  float* logit;
  int* list;
  unsigned* hist;
  float* red;
  float* tmp;     // 64 words: reduction scratch [0,32), broadcast [32,64)
  int* sel;
  __device__ AttnSmem(unsigned char* base, int rows) {
    const int cp = (rows + 3) & ~3;
    logit = reinterpret_cast<float*>(base);
    list = reinterpret_cast<int*>(logit + cp);
    hist = reinterpret_cast<unsigned*>(list + cp);
    red = reinterpret_cast<float*>(hist + 256);
    tmp = red + (NT / 32) * DH;
    sel = reinterpret_cast<int*>(tmp + 32);
  }
};

// Phases 2-3, given the logits of all C+1 rows in shared memory (-inf for empty slots): decides the
// kept set, turns the logits into weights in place (0 for rows not kept), writes the weights out and
// builds the ordered list of kept row indices. Returns the number of kept rows. Every thread of the
// block (scope SY) calls it after a barrier of that scope; the results are published by a final barrier.
//
// Every warp owns one contiguous segment of the rows and every lane keeps its rows' order-preserving keys in
// registers (row seg_begin + 32 k + lane in register k, KPT registers): the passes of the radix select, the maximum
// and the exponentials are then unrolled loops over registers with no shared-memory load in their dependency chains,
// and the kept rows are counted and placed with ballots; the block meets only to exchange counts.
template <typename T, int DH, int NT, int KPT, typename SY>
__device__ __forceinline__ int attention_keep_and_weights_impl(const AttnParams<T>& p, const AttnSmem<DH, NT>& sm, int bh, int seg) {
  constexpr int NW = NT / 32;
  float* s_logit = sm.logit;
  int* s_list = sm.list;
  unsigned* s_hist = sm.hist;
  float* s_tmp = sm.tmp;
  int* s_sel = sm.sel;
  const int rows = p.C + 1;
  const int tid = SY::tid(), lane = tid & 31, warp = tid >> 5;
  const int seg_begin = warp * seg, seg_end = min(rows, seg_begin + seg);

  // ---- phase 2: which logits are kept (K largest, lower index wins ties) -------------------
  uint32_t key[KPT];                      // 0 for positions past the segment: below every real key
  int cnt = 0;
#pragma unroll
  for (int k = 0; k < KPT; ++k) {
    const int i = seg_begin + 32 * k + lane;
    const float l = i < seg_end ? s_logit[i] : -INFINITY;
    key[k] = i < seg_end ? float_key(l) : 0u;
    cnt += (l > -INFINITY) ? 1 : 0;
  }
  for (int i = tid; i < 256; i += NT) s_hist[i] = 0u;
  const int n_cand = __float2int_rn(block_sum_f<NT, SY>(float(cnt), s_tmp));   // (its barriers also publish the zeroed bins)
  uint32_t thr_key = 0u;                  // keep every candidate unless there are more than K
  if (n_cand > p.topk) {
    uint32_t prefix = 0u, mask = 0u;
    int need = p.topk;
#pragma unroll
    for (int shift = 24; shift >= 0; shift -= 8) {
#pragma unroll
      for (int k = 0; k < KPT; ++k)
        if (key[k] != 0u && (key[k] & mask) == prefix) atomicAdd(&s_hist[(key[k] >> shift) & 255u], 1u);
      SY::sync();
      if (warp == 0) {
        int c[8], tot = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { c[j] = int(s_hist[lane * 8 + j]); tot += c[j]; s_hist[lane * 8 + j] = 0u; }   // bins ready for the next digit
        int incl = tot;                   // suffix sum: this lane's bins and all higher ones
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += t;
        }
        const int above = incl - tot;
        if (above < need && need <= above + tot) {
          int acc = above;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (acc < need && need <= acc + c[j]) { s_sel[0] = lane * 8 + j; s_sel[1] = need - acc; s_sel[2] = c[j]; }
            acc += c[j];
          }
        }
      }
      SY::sync();
      prefix |= uint32_t(s_sel[0]) << shift;
      mask |= 255u << shift;
      need = s_sel[1];
    }
    thr_key = prefix;
    const int n_eq = s_sel[2];
    if (n_eq != need) {                   // exact ties at the threshold (block-uniform): keep the lowest indices
      SY::sync();
      if (tid == 0) {
        int left = need;
        for (int i = 0; i < rows; ++i)
          if (float_key(s_logit[i]) == thr_key) { if (left > 0) --left; else s_logit[i] = -INFINITY; }
      }
      SY::sync();
#pragma unroll
      for (int k = 0; k < KPT; ++k) {     // the dropped rows now read -inf
        const int i = seg_begin + 32 * k + lane;
        if (i < seg_end) key[k] = float_key(s_logit[i]);
      }
    }
  }

  // ---- phase 3: softmax over the kept logits ----------------------------------------------
  // kept: a real key (float_key(-inf) = 0x007fffff and the padding 0 are below every finite logit's key) at or above the threshold
  constexpr uint32_t kMinusInfKey = 0x007fffffu;
  const uint32_t keep_from = thr_key > kMinusInfKey ? thr_key : kMinusInfKey + 1u;
  uint32_t kmax = 0u;
#pragma unroll
  for (int k = 0; k < KPT; ++k) kmax = (key[k] >= keep_from && key[k] > kmax) ? key[k] : kmax;
  // the largest key is the largest logit: undo the order-preserving map
  float mx = -INFINITY;
  if (kmax != 0u) mx = __uint_as_float((kmax & 0x80000000u) ? (kmax & 0x7fffffffu) : ~kmax);
  mx = block_max_f<NT, SY>(mx, s_tmp);
  float part = 0.f;
  int kept_here = 0;
  float ev[KPT];
#pragma unroll
  for (int k = 0; k < KPT; ++k) {
    const bool keep = key[k] >= keep_from;
    const float l = __uint_as_float((key[k] & 0x80000000u) ? (key[k] & 0x7fffffffu) : ~key[k]);
    ev[k] = keep ? expf(l - mx) : -1.f;   // -1 marks "not kept"
    part += keep ? ev[k] : 0.f;
    kept_here += __popc(__ballot_sync(0xffffffffu, keep));
  }
  if (lane == 0) s_sel[8 + warp] = kept_here;
  const float inv = 1.f / block_sum_f<NT, SY>(part, s_tmp);     // (its barriers also publish the warps' counts)
  int base = 0, n_kept = 0;
#pragma unroll
  for (int w = 0; w < NW; ++w) { const int c = s_sel[8 + w]; if (w < warp) base += c; n_kept += c; }
  // ordered compaction of the kept indices; weights replace the logits in place
#pragma unroll
  for (int k = 0; k < KPT; ++k) {
    const int i = seg_begin + 32 * k + lane;
    const bool keep = ev[k] >= 0.f;
    const unsigned bal = __ballot_sync(0xffffffffu, keep);
    const float wgt = keep ? ev[k] * inv : 0.f;
    if (i < seg_end) {
      s_logit[i] = wgt;
      if (p.weights) p.weights[size_t(bh) * rows + i] = wgt;
    }
    if (keep) s_list[base + __popc(bal & ((1u << lane) - 1u))] = i;
    base += __popc(bal);
  }
  SY::sync();
  return n_kept;
}

template <typename T, int DH, int NT = kAttnThreads, typename SY = CtaScope>
__device__ __forceinline__ int attention_keep_and_weights(const AttnParams<T>& p, const AttnSmem<DH, NT>& sm, int bh /* row of out/weights */) {
  constexpr int NW = NT / 32;
  const int rows = p.C + 1;
  const int seg = (((rows + NW - 1) / NW) + 31) & ~31;      // rows per warp, a multiple of 32
  // 9 registers per lane cover C <= 1151 with 4 warps and C <= 2303 with 8; kernels of 4 warps are launched for
  // C <= 1024 only, those of 8 warps for any capacity up to 4096 (17 registers)
  if (NT <= 128 || seg <= 9 * 32) return attention_keep_and_weights_impl<T, DH, NT, 9, SY>(p, sm, bh, seg);
  return attention_keep_and_weights_impl<T, DH, NT, 17, SY>(p, sm, bh, seg);
}

// Phase 4 with direct loads: adds w_s * V[s] of the kept rows [j_begin, n_kept) of the list into acc (this lane's 16-byte column
// slice; lanes of different row groups and warps hold partial sums). U loads of 16 bytes are in flight per lane: a gather of
// 256-byte rows needs on the order of 100 KB in flight per SM to run at the memory system's rate.
template <typename T, int DH, int NT = kAttnThreads, int U = kAttnUnroll, typename SY = CtaScope>
__device__ __forceinline__ void attention_values_direct(const AttnParams<T>& p, const AttnSmem<DH, NT>& sm, int bh, int n_kept,
                                                        float (&acc)[Elem<T>::kPer16B], int j_begin = 0) {
  constexpr int NW = NT / 32;
  constexpr int EPL = Elem<T>::kPer16B;
  constexpr int LPR = DH / EPL;
  constexpr int RPW = 32 / LPR;
  const float* s_logit = sm.logit;
  const int* s_list = sm.list;
  const int C = p.C;
  const int lane = SY::tid() & 31, warp = SY::tid() >> 5;
  const int sub = lane / LPR, li = lane % LPR;
  const size_t row_bytes = size_t(DH) * sizeof(T);
  const unsigned char* Vb = reinterpret_cast<const unsigned char*>(p.Vc) + size_t(bh) * C * row_bytes;
  const unsigned char* vnew = reinterpret_cast<const unsigned char*>(p.v_new) + size_t(bh) * row_bytes;
  // ---- phase 4: weighted sum of the kept value rows ----------------------------------------
  for (int j0 = j_begin + warp * RPW; j0 < n_kept; j0 += NW * RPW * U) {   // entries [j_begin, n_kept) of the kept list
    uint4 vv[U];
    float wv[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int j = j0 + u * NW * RPW + sub;
      vv[u] = make_uint4(0u, 0u, 0u, 0u);
      wv[u] = 0.f;
      if (j < n_kept) {
        const int idx = s_list[j];
        wv[u] = s_logit[idx];
        vv[u] = ldg_stream((idx == C ? vnew : Vb + size_t(idx) * row_bytes) + li * 16);
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      float vf[EPL];
      Elem<T>::unpack(vv[u], vf);
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[e] = fmaf(wv[u], vf[e], acc[e]);
    }
  }
}

// Adds the partial sums of all row groups and warps, writes `out`, then writes the current token's
// row into its slot (append of the most recent state, Section 2.2 third bullet).
template <typename T, int DH, int NT = kAttnThreads, typename SY = CtaScope>
__device__ __forceinline__ void attention_finish(const AttnParams<T>& p, const AttnSmem<DH, NT>& sm, int bh,
                                                 float (&acc)[Elem<T>::kPer16B], int out_row = -1, bool admit = true) {
  if (out_row < 0) out_row = bh;
  constexpr int NW = NT / 32;
  constexpr int EPL = Elem<T>::kPer16B;
  constexpr int LPR = DH / EPL;
  float* s_red = sm.red;
  const int C = p.C;
  const int tid = SY::tid(), lane = tid & 31, warp = tid >> 5;
  const int sub = lane / LPR, li = lane % LPR;
  const int b = bh / p.H;
  const size_t row_bytes = size_t(DH) * sizeof(T);
  unsigned char* Kb = reinterpret_cast<unsigned char*>(p.Kc) + size_t(bh) * C * row_bytes;
  unsigned char* Vb = reinterpret_cast<unsigned char*>(p.Vc) + size_t(bh) * C * row_bytes;
  const unsigned char* knew = reinterpret_cast<const unsigned char*>(p.k_new) + size_t(bh) * row_bytes;
  const unsigned char* vnew = reinterpret_cast<const unsigned char*>(p.v_new) + size_t(bh) * row_bytes;
#pragma unroll
  for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
  if (sub == 0)
#pragma unroll
    for (int e = 0; e < EPL; ++e) s_red[warp * DH + li * EPL + e] = acc[e];
  SY::sync();
  for (int e = tid; e < DH; e += NT) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) s += s_red[w * DH + e];
    p.out[size_t(out_row) * DH + e] = Elem<T>::from_float(s);
  }

  // ---- admit: the current token's row goes into its slot (all reads of this block are done) --
  if (admit && p.admit_slot != nullptr) {
    const int s = p.admit_slot[b];
    if (s >= 0 && s < C) {
      constexpr int V16 = int(sizeof(T)) * DH / 16;
      unsigned char* kd = Kb + size_t(s) * row_bytes;
      unsigned char* vd = Vb + size_t(s) * row_bytes;
      if (tid < V16) reinterpret_cast<uint4*>(kd)[tid] = reinterpret_cast<const uint4*>(knew)[tid];
      else if (tid < 2 * V16) reinterpret_cast<uint4*>(vd)[tid - V16] = reinterpret_cast<const uint4*>(vnew)[tid - V16];
    } else if (tid == 0) {
      set_error(p.err, ERRW_BOUNDS);
    }
  }
}

}  // namespace adore
