// Fused decode step of one layer: Section 2.2 attention of the G queries of every kv head
// over its slot-indexed cache (split-K over a persistent grid), and, by the CTA that
// completes a head last, Algorithm 1: top-p hit mask from the final softmax weights, CRF /
// tau update, lowest-CRF eviction with in-place slot reuse.
#pragma once
#include "common.cuh"
#include "evict.cuh"

namespace ckv {

template <int G>
struct Lay {
  static constexpr int PSTRIDE = G * (HD + 2);  // floats per split-K partial: m[G], l[G], O[G][128]
  static constexpr int MERGE_BYTES = NW * PSTRIDE * 4;
};

// ---------------------------------------------------------------------------------------
// Streaming side: one warp copies a group of 16 entries (K and V rows, 512 B each) into its
// ring slot with 16-byte cp.async, one full entry per warp instruction.
template <int G>
__device__ __forceinline__ void issue_group(const DecodeParams& p, int uid, int seq, int u_local,
                                            int n_tot, int n_old, int grp, unsigned char* slot,
                                            int lane) {
  const State& st = p.st;
  const int base = grp * GRP;
  const int valid = min(GRP, n_tot - base);
  const size_t mb = (size_t)uid * st.cap;
  const int my_slot = (lane < valid) ? st.list_slot[mb + base + lane] : 0;
  const unsigned char* poolseq = st.pool + (size_t)seq * st.slots_per_seq * SLOT_BYTES;
  const uint32_t sK = smem_u32(slot), sV = sK + K_REGION;
  const uint32_t dst0 = (lane < 16) ? sK + lane * 16 : sV + (lane - 16) * 16;
  const uint32_t dstep = (lane < 16) ? ROW_BYTES : V_STRIDE;
#pragma unroll
  for (int e = 0; e < GRP; ++e) {
    const int s = __shfl_sync(0xffffffffu, my_slot, e);
    const uint32_t dst = dst0 + e * dstep;
    if (e < valid) {
      unsigned char* row = const_cast<unsigned char*>(poolseq) + (size_t)s * SLOT_BYTES + lane * 16;
      if (p.append && base + e == n_old) {
        // the arriving token: take it from the call's inputs and store it in the head's spare slot
        const int head = uid % st.H;
        const __nv_bfloat16* src = (lane < 16 ? p.k_new : p.v_new) + ((size_t)seq * st.H + head) * HD;
        const uint4 val = *reinterpret_cast<const uint4*>(reinterpret_cast<const unsigned char*>(src) + (lane & 15) * 16);
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(dst), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
        *reinterpret_cast<uint4*>(row) = val;
        if (lane == 0) {
          st.meta_pos[mb + n_old] = p.t;
          st.meta_tau[mb + n_old] = p.t;
          st.meta_crf[mb + n_old] = 0.0f;
        }
      } else {
        cp_async16(dst, row);
      }
    } else {
      asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0) : "memory");
    }
  }
  cp_commit();
  (void)u_local;
}

// Running split-K state of one warp for the head it is streaming.
template <int G>
struct WarpAcc {
  float m[G];      // running max of scale*log2(e)*logit
  float l[G];      // lane-partial sum of exp2 (every key is held by two lanes)
  float O[G][8];   // lane-partial output: dims [8j, 8j+8) over the keys of this half-warp
  __device__ __forceinline__ void reset() {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      m[g] = -INFINITY;
      l[g] = 0.f;
#pragma unroll
      for (int d = 0; d < 8; ++d) O[g][d] = 0.f;
    }
  }
};

// One group of 16 keys: logits for the G queries (fp32 FMA, fixed summation order), online
// softmax, logits to the scratch for the hit mask, and P.V.
template <int G>
__device__ __forceinline__ void compute_group(const DecodeParams& p, const float (&qf)[G][8],
                                              WarpAcc<G>& acc, const unsigned char* slot, int valid,
                                              float* logit_row /* &logits[u][0][base] or null */,
                                              int lane) {
  const int half = lane >> 4, j = lane & 15, ml = j >> 1;
  const unsigned char* sK = slot;
  const unsigned char* sV = slot + K_REGION;
  float a[8][G];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int row = 2 * (i ^ ml) + half;
    const uint4 kk = *reinterpret_cast<const uint4*>(sK + row * ROW_BYTES + j * 16);
    const float kf[8] = {bf_lo(kk.x), bf_hi(kk.x), bf_lo(kk.y), bf_hi(kk.y),
                         bf_lo(kk.z), bf_hi(kk.z), bf_lo(kk.w), bf_hi(kk.w)};
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float s = qf[g][0] * kf[0];
#pragma unroll
      for (int d = 1; d < 8; ++d) s = fmaf(qf[g][d], kf[d], s);
      a[i][g] = s;
    }
  }
  // transpose-reduce over the 16 lanes of a row: lane j ends with key 2*(j>>1)+half
  float pg[G];
  const int e_mine = 2 * ml + half;
  const bool ok = e_mine < valid;
#pragma unroll
  for (int g = 0; g < G; ++g) {
    float r0 = a[0][g] + __shfl_xor_sync(0xffffffffu, a[4][g], 8);
    float r1 = a[1][g] + __shfl_xor_sync(0xffffffffu, a[5][g], 8);
    float r2 = a[2][g] + __shfl_xor_sync(0xffffffffu, a[6][g], 8);
    float r3 = a[3][g] + __shfl_xor_sync(0xffffffffu, a[7][g], 8);
    r0 += __shfl_xor_sync(0xffffffffu, r2, 4);
    r1 += __shfl_xor_sync(0xffffffffu, r3, 4);
    r0 += __shfl_xor_sync(0xffffffffu, r1, 2);
    r0 += __shfl_xor_sync(0xffffffffu, r0, 1);
    const float raw = r0;
    if (logit_row != nullptr && ok && (j & 1) == 0) logit_row[(size_t)g * p.sc.cap_s + e_mine] = __fmul_rn(raw, p.scale);
    float s2 = ok ? raw * p.scale_log2 : -INFINITY;
    float gm = s2;
#pragma unroll
    for (int o = 16; o > 1; o >>= 1) gm = fmaxf(gm, __shfl_xor_sync(0xffffffffu, gm, o));
    const float mn = fmaxf(acc.m[g], gm);
    if (mn > acc.m[g]) {  // warp-uniform
      const float corr = ex2(acc.m[g] - mn);
      acc.l[g] *= corr;
#pragma unroll
      for (int d = 0; d < 8; ++d) acc.O[g][d] *= corr;
      acc.m[g] = mn;
    }
    pg[g] = ex2(s2 - mn);
    acc.l[g] += pg[g];
  }
#pragma unroll
  for (int it = 0; it < 8; ++it) {
    const int row = 2 * it + half;
    const uint4 vv = *reinterpret_cast<const uint4*>(sV + row * V_STRIDE + j * 16);
    const float vf[8] = {bf_lo(vv.x), bf_hi(vv.x), bf_lo(vv.y), bf_hi(vv.y),
                         bf_lo(vv.z), bf_hi(vv.z), bf_lo(vv.w), bf_hi(vv.w)};
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float pp = __shfl_sync(0xffffffffu, pg[g], half * 16 + 2 * it);
#pragma unroll
      for (int d = 0; d < 8; ++d) acc.O[g][d] = fmaf(pp, vf[d], acc.O[g][d]);
    }
  }
}

// ---------------------------------------------------------------------------------------
// Finaliser, run by the CTA whose partial completed the head.
//
// Part A merges the split-K partials into `out`.  Part B is Algorithm 1 steps 1-4 for the
// head: exact per-query softmax of the stored logits (accurate expf, fixed reduction
// order), group-mean probability pbar, hit mask = smallest descending-pbar prefix whose
// exclusive mass is below p (ties in pbar by ascending position), CRF/tau update, eviction.
// The mass walk uses 2^-40 fixed-point integers so it is exact and order independent.
template <int G>
__device__ void finalise_unit(const DecodeParams& p, int uid, int seq, int head, int u_local,
                              int n, int npieces, unsigned char* shraw) {
  const State& st = p.st;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  constexpr int PS = Lay<G>::PSTRIDE;
  unsigned long long* hist = reinterpret_cast<unsigned long long*>(shraw);   // HIST_BINS u64
  float* redf = reinterpret_cast<float*>(shraw + HIST_BINS * 8);             // NW*8 floats
  unsigned long long* redu = reinterpret_cast<unsigned long long*>(redf + NW * 8);  // NW + 4
  float* s_m = reinterpret_cast<float*>(redu + NW + 4);                      // G
  float* s_l = s_m + 8;                                                      // G
  int* s_i = reinterpret_cast<int*>(s_l + 8);                                // 32 ints
  int* sh_ev = s_i + 32;                                                     // evict scratch (>= 300 ints)
  const size_t mb = (size_t)uid * st.cap;

  // ---- Part A: out = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m)
  {
    const float* part = p.sc.partials + (size_t)u_local * p.sc.pmax * PS;
    const int Hq = st.H * G;
    for (int idx = tid; idx < G * HD; idx += NT) {
      const int g = idx / HD, d = idx % HD;
      float mm = -INFINITY;
      for (int pc = 0; pc < npieces; ++pc) mm = fmaxf(mm, part[(size_t)pc * PS + g]);
      float L = 0.f, o = 0.f;
      for (int pc = 0; pc < npieces; ++pc) {
        const float sc = ex2(part[(size_t)pc * PS + g] - mm);
        L = fmaf(part[(size_t)pc * PS + G + g], sc, L);
        o = fmaf(part[(size_t)pc * PS + 2 * G + g * HD + d], sc, o);
      }
      p.out[((size_t)seq * Hq + head * G + g) * HD + d] = __float2bfloat16_rn(o / L);
    }
  }
  if (tid == 0) atomicAdd(&st.counters[0], (unsigned long long)n);
  int n_after = n;
  if (p.track) {
    const float* S = p.sc.logits + (size_t)u_local * G * p.sc.cap_s;
    float* pbar = p.sc.pbar + (size_t)u_local * p.sc.cap_s;
    // ---- step 1a: exact row max per query
    float mx[G];
#pragma unroll
    for (int g = 0; g < G; ++g) mx[g] = -INFINITY;
    for (int i = tid; i < n; i += NT)
#pragma unroll
      for (int g = 0; g < G; ++g) mx[g] = fmaxf(mx[g], S[(size_t)g * p.sc.cap_s + i]);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float v = warp_max(mx[g]);
      if (lane == 0) redf[w * 8 + g] = v;
    }
    __syncthreads();
    if (tid < G) {
      float v = redf[tid];
      for (int x = 1; x < NW; ++x) v = fmaxf(v, redf[x * 8 + tid]);
      s_m[tid] = v;
    }
    __syncthreads();
    // ---- step 1b: normalisers, summed in a fixed order
    float sm[G];
#pragma unroll
    for (int g = 0; g < G; ++g) { mx[g] = s_m[g]; sm[g] = 0.f; }
    for (int i = tid; i < n; i += NT)
#pragma unroll
      for (int g = 0; g < G; ++g) sm[g] += expf(S[(size_t)g * p.sc.cap_s + i] - mx[g]);
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
    // ---- step 1c: pbar_i = mean_g p_{g,i}; integer mass w_i = floor(pbar_i * 2^40)
    float li[G];
#pragma unroll
    for (int g = 0; g < G; ++g) li[g] = s_l[g];
    unsigned long long wsum = 0;
    for (int i = tid; i < n; i += NT) {
      float pm = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) pm += __fdiv_rn(expf(S[(size_t)g * p.sc.cap_s + i] - mx[g]), li[g]);
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
      if (tid == 0) s_i[0] = -1;
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
      // inclusive suffix scan across threads (higher tid = higher bins)
      unsigned long long suf = loc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned long long x = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += x;
      }
      if (lane == 0) redu[w] = suf;
      __syncthreads();
      unsigned long long above = 0;
      for (int x = w + 1; x < NW; ++x) above += redu[x];
      // mass above this thread's top bin
      unsigned long long sab = A + above + (suf - loc);
      for (int b = per - 1; b >= 0; --b) {
        const unsigned long long hb = hist[tid * per + b];
        if (sab < Pthr && Pthr <= sab + hb) {
          s_i[0] = tid * per + b;
          redu[NW] = sab;
        }
        sab += hb;
      }
      __syncthreads();
      const int dstar = s_i[0];
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
    if (lane == 0) s_i[4 + w] = eq;
    __syncthreads();
    int cnt_eq = 0;
    for (int x = 0; x < NW; ++x) cnt_eq += s_i[4 + x];
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
      __syncthreads();
      if (lane == 0) { s_i[8 + w * 4] = (int)bk0; s_i[9 + w * 4] = (int)bk1; s_i[10 + w * 4] = (int)bk2; s_i[11 + w * 4] = bidx; }
      __syncthreads();   // also orders every CRF/tau store above before the swap below
      if (tid == 0) {
        uint32_t m0 = (uint32_t)s_i[8], m1 = (uint32_t)s_i[9], m2 = (uint32_t)s_i[10];
        int mi = s_i[11];
        for (int x = 1; x < NW; ++x) {
          const uint32_t o0 = (uint32_t)s_i[8 + x * 4], o1 = (uint32_t)s_i[9 + x * 4], o2 = (uint32_t)s_i[10 + x * 4];
          const bool less = (o0 != m0) ? (o0 < m0) : ((o1 != m1) ? (o1 < m1) : (o2 < m2));
          if (less) { m0 = o0; m1 = o1; m2 = o2; mi = s_i[11 + x * 4]; }
        }
        // the leaving entry's slot becomes the head's spare at position n-1
        if (mi != n - 1) swap_into(st, mb, mi, n - 1);
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
  }
  if (n_after == n) {
    // nothing left the head: record the new length and fetch a fresh spare for position n
    if (tid == 0) {
      p.n_out[uid] = n;
      if (p.append) {
        if (n + 1 > st.cap) {
          atomicOr(st.errword, ERR_CAPACITY);
        } else {
          const int idx = atomicSub(&st.free_top[seq], 1) - 1;
          if (idx < 0) {
            atomicAdd(&st.free_top[seq], 1);
            atomicOr(st.errword, ERR_FREE_UNDERFLOW);
          } else {
            st.list_slot[mb + n] = st.free_stack[(size_t)seq * st.slots_per_seq + idx];
          }
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------
template <int G>
__global__ void __launch_bounds__(NT, (G <= 5 ? 3 : 2)) decode_kernel(const DecodeParams p) {
  extern __shared__ __align__(16) unsigned char smem[];
  unsigned char* ring = smem;                      // also the merge buffer and finaliser scratch
  int* off = reinterpret_cast<int*>(smem + RING_BYTES);   // U + 1 group prefix sums
  __shared__ int s_red[NW + 1];
  __shared__ int s_last;
  const State& st = p.st;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int U = st.batch * st.H;
  constexpr int PS = Lay<G>::PSTRIDE;

  // ---- every CTA derives the same flat split of all groups of this layer
  {
    int run = 0;
    for (int base = 0; base < U; base += NT) {
      const int u = base + tid;
      int g = 0;
      if (u < U) {
        const int uid = ((u / st.H) * st.L + p.layer) * st.H + (u % st.H);
        g = (p.n_in[uid] + p.append + GRP - 1) / GRP;
      }
      int tot;
      const int ex = block_excl_scan(g, s_red, tot);
      if (u < U) off[u] = run + ex;
      run += tot;
    }
    if (tid == 0) off[U] = run;
    __syncthreads();
  }
  const long long Gtot = off[U];
  if (Gtot == 0) return;
  const int nActive = (int)min((long long)gridDim.x, max(1ll, Gtot / GMIN));
  const int cta = blockIdx.x;
  if (cta >= nActive) return;
  const int lo = (int)((long long)cta * Gtot / nActive), hi = (int)((long long)(cta + 1) * Gtot / nActive);
  auto cta_of = [&](int x) {
    int c = (int)((long long)x * nActive / Gtot);
    while ((int)((long long)(c + 1) * Gtot / nActive) <= x) ++c;
    while ((int)((long long)c * Gtot / nActive) > x) --c;
    return c;
  };
  // first head whose group range contains `lo`
  int u = 0;
  {
    int a = 0, b = U;  // largest u with off[u] <= lo
    while (b - a > 1) {
      const int mid = (a + b) >> 1;
      if (off[mid] <= lo) a = mid; else b = mid;
    }
    u = a;
  }
  unsigned char* myring = ring + w * NSLOT * RING_SLOT_BYTES;
  const int half = lane >> 4, j = lane & 15;

  for (; u < U && off[u] < hi; ++u) {
    const int g0 = off[u], g1 = off[u + 1];
    if (g1 == g0) continue;
    const int a = max(lo, g0) - g0, b = min(hi, g1) - g0;   // this CTA's groups of head u
    const int seq = u / st.H, head = u % st.H;
    const int uid = (seq * st.L + p.layer) * st.H + head;
    const int n_old = p.n_in[uid];
    const int n_tot = n_old + p.append;
    // the G queries of this head: lane keeps dims [8j, 8j+8)
    float qf[G][8];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const uint4 qq = *reinterpret_cast<const uint4*>(
          reinterpret_cast<const unsigned char*>(p.q + ((size_t)seq * st.H * G + head * G + g) * HD) + j * 16);
      qf[g][0] = bf_lo(qq.x); qf[g][1] = bf_hi(qq.x); qf[g][2] = bf_lo(qq.y); qf[g][3] = bf_hi(qq.y);
      qf[g][4] = bf_lo(qq.z); qf[g][5] = bf_hi(qq.z); qf[g][6] = bf_lo(qq.w); qf[g][7] = bf_hi(qq.w);
    }
    WarpAcc<G> acc;
    acc.reset();
    const int cnt = (b - a > w) ? (b - a - w + NW - 1) / NW : 0;   // groups a+w, a+w+NW, ...
    float* lrow = p.track ? p.sc.logits + (size_t)u * G * p.sc.cap_s : nullptr;
    if (cnt > 0) issue_group<G>(p, uid, seq, u, n_tot, n_old, a + w, myring, lane);
    for (int k = 0; k < cnt; ++k) {
      const int grp = a + w + k * NW;
      if (k + 1 < cnt) {
        issue_group<G>(p, uid, seq, u, n_tot, n_old, grp + NW, myring + ((k + 1) & 1) * RING_SLOT_BYTES, lane);
        cp_wait<1>();
      } else {
        cp_wait<0>();
      }
      __syncwarp();
      compute_group<G>(p, qf, acc, myring + (k & 1) * RING_SLOT_BYTES, min(GRP, n_tot - grp * GRP),
                       lrow ? lrow + grp * GRP : nullptr, lane);
      __syncwarp();
    }
    // ---- merge the CTA's warps, publish the partial, take a ticket
    __syncthreads();   // every warp is done with its ring: reuse it as the merge buffer
    float* mbuf = reinterpret_cast<float*>(ring);
    {
      float* mine = mbuf + w * PS;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        const float lsum = warp_sum(acc.l[g]) * 0.5f;
        if (lane == 0) { mine[g] = acc.m[g]; mine[G + g] = lsum; }
#pragma unroll
        for (int d = 0; d < 8; ++d) {
          const float o = acc.O[g][d] + __shfl_xor_sync(0xffffffffu, acc.O[g][d], 16);
          if (half == 0) mine[2 * G + g * HD + j * 8 + d] = o;
        }
      }
    }
    __syncthreads();
    const int c_first = cta_of(g0), c_last = cta_of(g1 - 1);
    const int piece = cta - c_first, npieces = c_last - c_first + 1;
    float* part = p.sc.partials + ((size_t)u * p.sc.pmax + piece) * PS;
    for (int idx = tid; idx < G * HD; idx += NT) {
      const int g = idx / HD;
      float mm = -INFINITY;
#pragma unroll
      for (int x = 0; x < NW; ++x) mm = fmaxf(mm, mbuf[x * PS + g]);
      float o = 0.f;
#pragma unroll
      for (int x = 0; x < NW; ++x) {
        const float mw = mbuf[x * PS + g];
        if (mw > -INFINITY) o = fmaf(mbuf[x * PS + 2 * G + idx], ex2(mw - mm), o);
      }
      part[2 * G + idx] = o;
    }
    if (tid < G) {
      float mm = -INFINITY;
#pragma unroll
      for (int x = 0; x < NW; ++x) mm = fmaxf(mm, mbuf[x * PS + tid]);
      float l = 0.f;
#pragma unroll
      for (int x = 0; x < NW; ++x) {
        const float mw = mbuf[x * PS + tid];
        if (mw > -INFINITY) l = fmaf(mbuf[x * PS + G + tid], ex2(mw - mm), l);
      }
      part[tid] = mm;
      part[G + tid] = l;
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const int old = atomicAdd(&p.sc.ticket[u], 1);
      s_last = (old == npieces - 1);
      if (s_last) p.sc.ticket[u] = 0;   // ready for the next launch
    }
    __syncthreads();
    if (s_last) {
      __threadfence();
      finalise_unit<G>(p, uid, seq, head, u, n_tot, npieces, ring);
    }
    __syncthreads();
  }
}

}  // namespace ckv
