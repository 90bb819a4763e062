// Algorithm 1 for the heads of one layer, one CTA per head, from the scaled logits the
// attention kernel left in the scratch (the cache itself is not read again):
//   step 1   exact softmax per query head (accurate expf, fixed reduction order), group-mean
//            probability pbar, hit mask = smallest descending-pbar prefix whose exclusive
//            mass is below p (equal pbar: ascending position);
//   step 2-3 hits: CRF <- lambda^(t - tau) CRF + 1, tau <- t; misses only get the decayed
//            CRF_temp, which is not stored;
//   step 4   the entries lowest under (CRF_temp, tau, position) leave until the head is
//            within its budget; the freed slot is reused in place.
// The mass walk uses 2^-40 fixed-point integers so it is exact and order independent.
#pragma once
#include "common.cuh"
#include "evict.cuh"

namespace ckv {

constexpr int HIST_BINS = 2048;

template <int G>
__global__ void __launch_bounds__(NT) lrfu_kernel(const DecodeParams p) {
  __shared__ unsigned long long hist[HIST_BINS];
  __shared__ float redf[NW * 8];
  __shared__ unsigned long long redu[NW + 4];
  __shared__ float s_l[8];
  __shared__ int s_star;
  __shared__ int s_eq[NW];
  __shared__ int s_min[NW * 4];
  __shared__ int sh_ev[320];
  const State& st = p.st;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + p.layer) * st.H + head;
  const size_t mb = (size_t)uid * st.cap;
  const int n = p.n_in[uid] + p.append;
  if (n <= 0) {
    if (tid == 0) p.n_out[uid] = 0;
    return;
  }
  const float* S = p.sc.logits + (size_t)u * p.sc.cap_s * QH;
  float* pbar = p.sc.pbar + (size_t)u * p.sc.cap_s;

  // ---- step 1a: normalisers, shifted by the attention kernel's running maximum
  float mx[G], sm[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    mx[g] = p.sc.mfin[u * QH + g] * 0.693147180559945309f;   // log2 domain -> natural log
    sm[g] = 0.f;
  }
  for (int i = tid; i < n; i += NT) {
    const float4 a = *reinterpret_cast<const float4*>(S + (size_t)i * QH);
    const float4 b = *reinterpret_cast<const float4*>(S + (size_t)i * QH + 4);
    const float sv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int g = 0; g < G; ++g) sm[g] += expf(sv[g] - mx[g]);
  }
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const float v = warp_sum(sm[g]);
    if (lane == 0) redf[w * 8 + g] = v;
  }
  __syncthreads();
  if (tid < G) {
    float v = redf[tid];
    for (int x = 1; x < NW; ++x) v += redf[x * 8 + tid];
    s_l[tid] = v;
  }
  __syncthreads();
  // ---- step 1b: pbar_i = mean_g p_{g,i}; integer mass w_i = floor(pbar_i * 2^40)
  float li[G];
#pragma unroll
  for (int g = 0; g < G; ++g) li[g] = s_l[g];
  unsigned long long wsum = 0;
  for (int i = tid; i < n; i += NT) {
    const float4 a = *reinterpret_cast<const float4*>(S + (size_t)i * QH);
    const float4 b = *reinterpret_cast<const float4*>(S + (size_t)i * QH + 4);
    const float sv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float pm = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) pm += __fdiv_rn(expf(sv[g] - mx[g]), li[g]);
    pm = __fdiv_rn(pm, (float)G);
    pbar[i] = pm;
    wsum += (unsigned long long)(pm * 1099511627776.0f);
  }
  wsum = warp_sum_u64(wsum);
  if (lane == 0) redu[w] = wsum;
  __syncthreads();
  unsigned long long W = 0;
  for (int x = 0; x < NW; ++x) W += redu[x];
  // hit  <=>  mass strictly before the entry  <  p * W
  const unsigned long long Pthr = (unsigned long long)ceil((double)p.top_p * (double)W);
  // ---- threshold key by MSB-first radix passes over the fp32 bits of pbar (11, 11, 10 bits)
  unsigned long long A = 0;   // mass of keys strictly above the current prefix range
  uint32_t prefix = 0;
  bool found_all = true;
  const int shifts[3] = {21, 10, 0};
  const int widths[3] = {11, 11, 10};
  for (int pass = 0; pass < 3; ++pass) {
    const int sh = shifts[pass], nb = 1 << widths[pass];
    __syncthreads();
    for (int b = tid; b < nb; b += NT) hist[b] = 0ull;
    if (tid == 0) s_star = -1;
    __syncthreads();
    for (int i = tid; i < n; i += NT) {
      const float pm = pbar[i];
      const uint32_t key = __float_as_uint(pm);
      const bool match = (pass == 0) || ((key >> (sh + widths[pass])) == (prefix >> (sh + widths[pass])));
      if (match) atomicAdd(&hist[(key >> sh) & (nb - 1)], (unsigned long long)(pm * 1099511627776.0f));
    }
    __syncthreads();
    // suffix sums from the top bin: thread k owns bins [k*per, (k+1)*per)
    const int per = nb / NT;
    unsigned long long loc = 0;
    for (int b = 0; b < per; ++b) loc += hist[tid * per + b];
    unsigned long long suf = loc;   // inclusive suffix scan across the warp (higher lane = higher bins)
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long x = __shfl_down_sync(0xffffffffu, suf, o);
      if (lane + o < 32) suf += x;
    }
    if (lane == 0) redu[w] = suf;
    __syncthreads();
    unsigned long long above = 0;
    for (int x = w + 1; x < NW; ++x) above += redu[x];
    unsigned long long sab = A + above + (suf - loc);   // mass above this thread's top bin
    for (int b = per - 1; b >= 0; --b) {
      const unsigned long long hb = hist[tid * per + b];
      if (sab < Pthr && Pthr <= sab + hb) {
        s_star = tid * per + b;
        redu[NW] = sab;
      }
      sab += hb;
    }
    __syncthreads();
    const int dstar = s_star;
    if (dstar < 0) { found_all = false; break; }
    prefix |= (uint32_t)dstar << sh;
    A = redu[NW];
  }
  __syncthreads();
  if (!found_all) {
    if (tid == 0) atomicOr(st.errword, ERR_NUCLEUS);
    prefix = 0xffffffffu;  // nothing is a hit
  }
  // ---- entries whose pbar equals the threshold key share one mass; the earliest positions win
  const uint32_t theta = prefix;
  int eq = 0;
  for (int i = tid; i < n; i += NT) eq += (__float_as_uint(pbar[i]) == theta);
  eq = warp_sum_i(eq);
  if (lane == 0) s_eq[w] = eq;
  __syncthreads();
  int cnt_eq = 0;
  for (int x = 0; x < NW; ++x) cnt_eq += s_eq[x];
  const unsigned long long w_theta = (unsigned long long)(__uint_as_float(theta) * 1099511627776.0f);
  // ---- steps 2-3: CRF/tau update; step 4 candidates
  const int k_evict = n - st.budget[uid];
  uint32_t bk0 = 0xffffffffu, bk1 = 0xffffffffu, bk2 = 0xffffffffu;
  int bidx = -1, nhit = 0;
  for (int i = tid; i < n; i += NT) {
    const uint32_t key = __float_as_uint(pbar[i]);
    bool hit = key > theta && found_all;
    const int pos_i = st.meta_pos[mb + i];
    if (key == theta && found_all) {
      unsigned long long rank = 0;
      if (cnt_eq > 1)
        for (int x = 0; x < n; ++x)
          rank += (__float_as_uint(pbar[x]) == theta) && (st.meta_pos[mb + x] < pos_i);
      hit = (A + rank * w_theta) < Pthr;
    }
    int tau = st.meta_tau[mb + i];
    float ct = __fmul_rn(st.tab[p.t - tau], st.meta_crf[mb + i]);
    if (hit) {
      ct = __fadd_rn(ct, 1.0f);
      tau = p.t;
      st.meta_crf[mb + i] = ct;
      st.meta_tau[mb + i] = tau;
      ++nhit;
    }
    if (k_evict == 1) {
      const uint32_t c0 = __float_as_uint(ct), c1 = (uint32_t)tau, c2 = (uint32_t)pos_i;
      const bool less = (c0 != bk0) ? (c0 < bk0) : ((c1 != bk1) ? (c1 < bk1) : (c2 < bk2));
      if (less) { bk0 = c0; bk1 = c1; bk2 = c2; bidx = i; }
    }
  }
  nhit = warp_sum_i(nhit);
  if (lane == 0 && nhit) atomicAdd(&st.counters[1], (unsigned long long)nhit);
  int n_after = n;
  if (k_evict == 1) {
    // block argmin of (CRF_temp, tau, pos)
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const uint32_t o0 = __shfl_xor_sync(0xffffffffu, bk0, o), o1 = __shfl_xor_sync(0xffffffffu, bk1, o),
                     o2 = __shfl_xor_sync(0xffffffffu, bk2, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bidx, o);
      const bool less = (o0 != bk0) ? (o0 < bk0) : ((o1 != bk1) ? (o1 < bk1) : (o2 < bk2));
      if (less) { bk0 = o0; bk1 = o1; bk2 = o2; bidx = oi; }
    }
    if (lane == 0) { s_min[w * 4] = (int)bk0; s_min[w * 4 + 1] = (int)bk1; s_min[w * 4 + 2] = (int)bk2; s_min[w * 4 + 3] = bidx; }
    __syncthreads();   // also orders every CRF/tau store above before the swap below
    if (tid == 0) {
      uint32_t a0 = (uint32_t)s_min[0], a1 = (uint32_t)s_min[1], a2 = (uint32_t)s_min[2];
      int ai = s_min[3];
      for (int x = 1; x < NW; ++x) {
        const uint32_t o0 = (uint32_t)s_min[x * 4], o1 = (uint32_t)s_min[x * 4 + 1], o2 = (uint32_t)s_min[x * 4 + 2];
        const bool less = (o0 != a0) ? (o0 < a0) : ((o1 != a1) ? (o1 < a1) : (o2 < a2));
        if (less) { a0 = o0; a1 = o1; a2 = o2; ai = s_min[x * 4 + 3]; }
      }
      // the leaving entry's slot becomes the head's spare at position n-1
      if (ai != n - 1) swap_into(st, mb, ai, n - 1);
      p.n_out[uid] = n - 1;
      atomicAdd(&st.counters[2], 1ull);
    }
    n_after = n - 1;
  } else if (k_evict > 1) {
    __syncthreads();
    if (p.append && tid == 0) atomicOr(st.errword, ERR_OVER_EVICT);
    evict_many(st, p.n_out, uid, seq, n, min(k_evict, n - 1), p.t, p.release != 0, sh_ev,
               reinterpret_cast<int*>(pbar));
    n_after = n - min(k_evict, n - 1);
  }
  if (n_after == n && tid == 0) keep_and_refill(st, p.n_out, uid, seq, n, p.append != 0);
}

}  // namespace ckv
