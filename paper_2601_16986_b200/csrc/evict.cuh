// Algorithm 1 step 4 for the cases in which several entries leave a head at once (a prompt longer
// than the budget, a budget that shrank, a buffered eviction cadence): pick the k entries lowest
// under (CRF decayed to now, tau, position) by a radix select, then close the gaps they leave by
// moving at most k entries from the end of the list into them (their rows and their metadata), so
// that the list is dense again and the pages past its end can go back to the sequence's free
// list.  (A decode step in which one entry leaves moves nothing: the arriving token of the next
// step takes the leaver's place.)
#pragma once
#include "common.cuh"

namespace ckv {

struct Key96 {
  uint32_t w[3];  // CRF_temp bits (>= +0, so unsigned order == float order), tau, pos
};

__device__ __forceinline__ Key96 entry_key(const State& st, size_t mb, int i, int t) {
  Key96 k;
  const int tau = st.meta_tau[mb + i];
  // lambda^(t - tau) * CRF, one fp32 rounding (Algorithm 1 steps 2-3 before the "+ 1")
  k.w[0] = __float_as_uint(__fmul_rn(st.tab[t - tau], st.meta_crf[mb + i]));
  k.w[1] = static_cast<uint32_t>(tau);
  k.w[2] = static_cast<uint32_t>(st.meta_pos[mb + i]);
  return k;
}

__device__ __forceinline__ bool key_le(const Key96& a, const uint32_t* b) {
  if (a.w[0] != b[0]) return a.w[0] < b[0];
  if (a.w[1] != b[1]) return a.w[1] < b[1];
  return a.w[2] <= b[2];
}

// Moves the entry at list position `src` of a head to position `dst` (one warp: lane c carries
// chunk c of the 512-byte row, which sits at a different place in the two pages' layouts).
__device__ __forceinline__ void move_entry(const State& st, int uid, int seq, size_t mb, int dst, int src, int lane,
                                           bool rows = true) {
  if (rows) {
    const uint4 v = *reinterpret_cast<const uint4*>(entry_chunk(st, uid, seq, src, lane));
    *reinterpret_cast<uint4*>(entry_chunk(st, uid, seq, dst, lane)) = v;
  }
  if (lane == 0) {
    st.meta_pos[mb + dst] = st.meta_pos[mb + src];
    st.meta_tau[mb + dst] = st.meta_tau[mb + src];
    st.meta_crf[mb + dst] = st.meta_crf[mb + src];
  }
}

// The pages a head owns beyond those that back list positions 0 .. n_new return to the
// sequence's free list.  Only called from launches in which no head takes a page.
__device__ __forceinline__ void release_pages(const State& st, int uid, int seq, int n_new, int* s_base) {
  const int need = n_new / GRP + 1;   // position n_new (the hole) stays backed
  const int have = st.npages[uid];
  const int cnt = have - need;
  if (cnt <= 0) return;
  if (threadIdx.x == 0) *s_base = atomicAdd(&st.free_top[seq], cnt);
  __syncthreads();
  const int base = *s_base;
  int* stack = st.free_stack + (size_t)seq * st.pages_per_seq;
  for (int r = threadIdx.x; r < cnt; r += NT) stack[base + r] = st.ptab[(size_t)uid * st.capg + need + r];
  __syncthreads();
  if (threadIdx.x == 0) st.npages[uid] = need;
}

// Removes the k lowest entries (1 <= k < n) of head `uid` at time t; the head's n entries must be
// dense (list positions 0 .. n-1).  `sh` is >= 1.2 KB (300 ints) of shared scratch, `tmp` a global
// int scratch of >= n words.  rows = false: the entries have no rows in the pool yet (a prompt
// that is being scored), only their metadata moves.  All NT threads call it.
__device__ void evict_many(const State& st, int uid, int seq, int n, int k, int t, bool release, int* sh, int* tmp,
                           bool rows = true) {
  const size_t mb = (size_t)uid * st.cap;
  int* hist = sh;             // 256
  int* s_kw = sh + 256;       // 3 words of the k-th key
  int* s_krem = sh + 259;
  int* red = sh + 260;        // NW + 1
  const int tid = threadIdx.x;
  int* s_done = sh + 260 + NW + 1;
  if (tid < 3) s_kw[tid] = 0;
  if (tid == 0) { *s_krem = k; *s_done = 0; }
  __syncthreads();
  // MSB-first radix select of the k-th smallest 96-bit key, 8 bits per pass.  The search stops
  // as soon as every entry that shares the prefix found so far is among the k lowest: the
  // prefix followed by all ones then separates the same set as the k-th key itself.
  for (int word = 0; word < 3 && !*s_done; ++word) {
    for (int shift = 24; shift >= 0 && !*s_done; shift -= 8) {
      for (int b = tid; b < 256; b += NT) hist[b] = 0;
      __syncthreads();
      const uint32_t k0 = s_kw[0], k1 = s_kw[1], k2 = s_kw[2];
      const uint32_t kw[3] = {k0, k1, k2};
      for (int i = tid; i < n; i += NT) {
        const Key96 key = entry_key(st, mb, i, t);
        bool match = true;
        for (int x = 0; x < word; ++x) match = match && (key.w[x] == kw[x]);
        if (shift < 24) match = match && ((key.w[word] >> (shift + 8)) == (kw[word] >> (shift + 8)));
        if (match) atomicAdd(&hist[(key.w[word] >> shift) & 255u], 1);
      }
      __syncthreads();
      if (tid < 32) {
        int loc = 0;
#pragma unroll
        for (int b = 0; b < 8; ++b) loc += hist[tid * 8 + b];
        int inc = loc;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int x = __shfl_up_sync(0xffffffffu, inc, o);
          if (tid >= o) inc += x;
        }
        const int krem = *s_krem;
        const int before = inc - loc;
        if (before < krem && krem <= inc) {  // exactly one lane
          int cum = before;
          for (int b = 0; b < 8; ++b) {
            const int c = hist[tid * 8 + b];
            if (cum + c >= krem) {
              uint32_t found = kw[word] | (static_cast<uint32_t>(tid * 8 + b) << shift);
              if (krem - cum == c) {   // the whole bucket leaves
                found |= (shift > 0) ? ((1u << shift) - 1u) : 0u;
                for (int x = word + 1; x < 3; ++x) s_kw[x] = static_cast<int>(0xffffffffu);
                *s_done = 1;
              }
              s_kw[word] = static_cast<int>(found);
              *s_krem = krem - cum;
              break;
            }
            cum += c;
          }
        }
      }
      __syncthreads();
    }
  }
  const uint32_t kth[3] = {(uint32_t)s_kw[0], (uint32_t)s_kw[1], (uint32_t)s_kw[2]};
  const int nk = n - k;
  // gaps: leaving entries inside the surviving range [0, nk)
  int gaps = 0;
  for (int base = 0; base < nk; base += NT) {
    const int i = base + tid;
    const int flag = (i < nk) && key_le(entry_key(st, mb, i, t), kth);
    int tot;
    const int r = block_excl_scan(flag, red, tot);
    if (flag) tmp[gaps + r] = i;
    gaps += tot;
  }
  // movers: staying entries in the tail [nk, n), as many as there are gaps
  int movers = 0;
  for (int base = nk; base < n; base += NT) {
    const int i = base + tid;
    const int flag = (i < n) && !key_le(entry_key(st, mb, i, t), kth);
    int tot;
    const int r = block_excl_scan(flag, red, tot);
    if (flag) tmp[gaps + movers + r] = i;
    movers += tot;
  }
  __syncthreads();
  // every mover fills one gap, in order; rows and metadata travel together
  for (int j = tid >> 5; j < min(gaps, movers); j += NW) move_entry(st, uid, seq, mb, tmp[j], tmp[gaps + j], tid & 31, rows);
  __syncthreads();
  if (tid == 0) {
    st.n_cur[uid] = nk;
    st.hole[uid] = nk;
    atomicAdd(&st.counters[2], (unsigned long long)k);
  }
  if (release && rows) release_pages(st, uid, seq, nk, s_krem);
}

}  // namespace ckv
