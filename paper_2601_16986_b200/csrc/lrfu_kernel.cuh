// Algorithm 1 for the heads of one layer, one CTA per head, from the scaled logits the
// attention kernel left in the scratch (the cache itself is not read again):
//   step 1   softmax weights per query head from the logits, the attention kernel's merged
//            reference point and normaliser (accurate expf), group-mean probability pbar,
//            hit mask = smallest descending-pbar prefix whose exclusive mass is below p
//            (equal pbar: ascending position).  The threshold value is found exactly: one
//            histogram of 1024 bins of 1/64 octave around 1/n locates its bin, the few
//            entries of that bin are ranked against one another; a bin outside the window
//            or with more than 64 entries falls back to four 8-bit radix passes over all bits;
//   step 2-3 hits: CRF <- lambda^(t - tau) CRF + 1, tau <- t; misses only get the decayed
//            CRF_temp, which is not stored;
//   step 4   the entries lowest under (CRF_temp, tau, position) leave until the head is
//            within its budget; the place of a single leaver becomes the head's hole, which
//            the next arriving token fills: nothing is moved.
// A launch without Algorithm 1 (answer stage, full-cache mode) only lets every head keep its new
// entry.  Either way the CTA that finishes last writes the layer's next launch plan (plan.cuh) when
// a head's length has drifted from the one the current plan was made for.
// The mass walk uses 2^-40 fixed-point integers so it is exact and order independent; the
// threshold is relative to the integer total, so a common factor on pbar changes nothing.
#pragma once
#include "common.cuh"
#include "evict.cuh"
#include "plan.cuh"

namespace ckv {

constexpr int HIST_BINS = 1024;   // shared histogram size: the fine pass uses all of it, a radix pass 256
constexpr float MASS_ONE = 1099511627776.0f;   // 2^40

constexpr int FINE_BINS = 1024;   // fast path: bins of 2^17 key steps = 1/64 octave, 16 octaves wide
constexpr int FINE_SHIFT = 17;
constexpr int MAX_CAND = 64;

struct LrfuSmem {
  unsigned hist_lo[HIST_BINS];   // per-bin mass, low 16 bits of every term
  unsigned hist_hi[HIST_BINS];   // per-bin mass, the bits above
  unsigned long long redu[NW + 4];
  unsigned cand[MAX_CAND];       // keys of the entries in the threshold's bin
  unsigned long long A_theta;    // fast path result: mass strictly above the threshold key
  unsigned theta;                //                   the threshold key
  int cnt_theta;                 //                   entries that carry it
  int ncand;
  int star;
  int eq[NW];
  int amin[NW * 4];
  int ev[320];
  int is_last;
};
static_assert(sizeof(LrfuSmem) >= (MAX_UNITS_PER_CALL + 1) * sizeof(int) + 321 * sizeof(int), "the planner's prefix sums reuse this memory");

// Loads the compiler must leave where they are written: the kernel is bound by the latency of
// its dependent global reads (several microseconds each while the attention kernel saturates
// HBM), so every read whose address is known is requested up front, in one batch.
__device__ __forceinline__ int ld_i32(const int* p) {
  int v;
  asm volatile("ld.global.b32 %0, [%1];\n" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float ld_f32(const float* p) {
  float v;
  asm volatile("ld.global.f32 %0, [%1];\n" : "=f"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ float4 ld_f32x4(const float* p) {
  float4 v;
  asm volatile("ld.global.v4.f32 {%0,%1,%2,%3}, [%4];\n" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
  return v;
}

constexpr int FRONT = 5;   // entries per thread whose logit rows are requested before n is known

// What the kernel requests before it knows the head's length.
template <int G>
struct Front {
  float4 ra[FRONT], rb[FRONT];   // logit rows of entries tid, tid + NT, ... (index clamped to the scratch)
  float m[G], l[G];              // merged reference point (log2 domain) and normaliser per query head
  int budget;
};

__device__ __forceinline__ unsigned long long mass_of(float pm) { return (unsigned long long)(pm * MASS_ONE); }

// EPT > 0: every thread keeps the pbar of its entries tid, tid + NT, ... (at most EPT) in
// registers; EPT == 0: they live in the global scratch and any n is allowed.
template <int G, int EPT>
__device__ int lrfu_unit(const DecodeParams& p, int u, int uid, int seq, int n, LrfuSmem& sh, const Front<G>& fr) {
  constexpr int R = EPT > 0 ? EPT : 1;
  const State& st = p.st;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const size_t mb = (size_t)uid * st.cap;
  const float* S = p.sc.logits + (size_t)u * p.sc.cap_s * QH;
  float* pbar = p.sc.pbar + (size_t)u * p.sc.cap_s;
  const int kmax = EPT > 0 ? (n + NT - 1) / NT : 0;

  // ---- step 1: pbar_i = mean_g exp(s_gi - m_g) / l_g
  float mx[G], invl[G];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    mx[g] = fr.m[g] * 0.693147180559945309f;   // log2 domain -> natural log
    invl[g] = 1.0f / (fr.l[g] * (float)G);
  }
  auto pbar_of = [&](int i) {
    const float4 a = *reinterpret_cast<const float4*>(S + (size_t)i * QH);
    float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
    if (G > 4) b = *reinterpret_cast<const float4*>(S + (size_t)i * QH + 4);
    const float sv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    float pm = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) pm = fmaf(expf(sv[g] - mx[g]), invl[g], pm);
    return pm;
  };
  float pmr[R];
  // stored state of this thread's entries, requested as soon as the logits are consumed so that
  // the reads complete under the threshold search (EPT == FRONT only)
  int pos_r[R], tau_r[R];
  float crf_r[R];
  if (EPT == FRONT) {
#pragma unroll
    for (int k = 0; k < R; ++k) {
      const float sv[8] = {fr.ra[k].x, fr.ra[k].y, fr.ra[k].z, fr.ra[k].w, fr.rb[k].x, fr.rb[k].y, fr.rb[k].z, fr.rb[k].w};
      float pm = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) pm = fmaf(expf(sv[g] - mx[g]), invl[g], pm);
      pmr[k] = (tid + k * NT < n) ? pm : 0.f;
    }
#pragma unroll
    for (int k = 0; k < R; ++k) {
      const size_t i = mb + min(tid + k * NT, n - 1);
      pos_r[k] = ld_i32(st.meta_pos + i);
      tau_r[k] = ld_i32(st.meta_tau + i);
      crf_r[k] = ld_f32(st.meta_crf + i);
    }
    // The logit rows are dead now (every thread holds its own in registers since before the
    // kernel learnt n, and nothing reads them again): drop their L2 lines instead of letting
    // them be written back to DRAM later.  Four 32-byte rows share a 128-byte line; units start
    // on line boundaries (cap_s is a multiple of four).
    // The barrier takes a value computed from every pbar, so no thread passes it with a row
    // load still in flight.
    int unordered = 0;
#pragma unroll
    for (int k = 0; k < R; ++k) unordered |= (pmr[k] != pmr[k]);
    (void)__syncthreads_or(unordered);
    if ((tid & 3) == 0) {
#pragma unroll
      for (int k = 0; k < R; ++k) {
        const int i = tid + k * NT;
        if (i < n) asm volatile("discard.global.L2 [%0], 128;\n" ::"l"(S + (size_t)i * QH) : "memory");
      }
    }
  } else if (EPT > 0) {
    // batches of BR entries whose rows are requested together (clamped index, no branch): while the
    // attention kernel saturates HBM every dependent round of loads costs this CTA microseconds, so
    // a batch is as large as the registers allow (only the G logits of a row are loaded)
    constexpr int BR = G <= 5 ? 8 : 4;
#pragma unroll
    for (int k = 0; k < R; ++k) pmr[k] = 0.f;
#pragma unroll
    for (int k0 = 0; k0 < R; k0 += BR) {
      if (k0 < kmax) {
        float4 ra[BR];
        float rb[BR][4];
#pragma unroll
        for (int j = 0; j < BR; ++j) {
          const int i = min(tid + (k0 + j) * NT, n - 1);
          ra[j] = ld_f32x4(S + (size_t)i * QH);
          if (G == 5) {
            rb[j][0] = ld_f32(S + (size_t)i * QH + 4);
          } else if (G > 5) {
            const float4 t4 = ld_f32x4(S + (size_t)i * QH + 4);
            rb[j][0] = t4.x; rb[j][1] = t4.y; rb[j][2] = t4.z; rb[j][3] = t4.w;
          }
        }
#pragma unroll
        for (int j = 0; j < BR; ++j) {
          if (k0 + j < R) {
            const float sv[8] = {ra[j].x, ra[j].y, ra[j].z, ra[j].w, G > 4 ? rb[j][0] : 0.f, G > 5 ? rb[j][1] : 0.f,
                                 G > 6 ? rb[j][2] : 0.f, G > 7 ? rb[j][3] : 0.f};
            float pm = 0.f;
#pragma unroll
            for (int g = 0; g < G; ++g) pm = fmaf(expf(sv[g] - mx[g]), invl[g], pm);
            pmr[k0 + j] = (tid + (k0 + j) * NT < n) ? pm : 0.f;
          }
        }
      }
    }
  } else {
    for (int i = tid; i < n; i += NT) pbar[i] = pbar_of(i);
  }
  // ---- fast path, pass over all entries: histogram of mass in fine bins around 1/n
  //      bin(key) = clamp((key >> 17) - base, 0, 1023), monotone in key
  const int fbase = (int)(__float_as_uint(1.0f / (256.0f * (float)n)) >> FINE_SHIFT);
  auto fbin = [&](uint32_t key) { return min(FINE_BINS - 1, max(0, (int)(key >> FINE_SHIFT) - fbase)); };
  for (int b = tid; b < FINE_BINS; b += NT) { sh.hist_lo[b] = 0u; sh.hist_hi[b] = 0u; }
  if (tid == 0) { sh.star = -1; sh.ncand = 0; sh.theta = 0xffffffffu; sh.cnt_theta = 0; }
  __syncthreads();
  {
    auto add = [&](float pm) {
      const unsigned long long m = mass_of(pm);
      const int b = fbin(__float_as_uint(pm));
      atomicAdd(&sh.hist_lo[b], (unsigned)(m & 0xffffu));
      atomicAdd(&sh.hist_hi[b], (unsigned)(m >> 16));
    };
    if (EPT > 0) {
#pragma unroll
      for (int k = 0; k < R; ++k)
        if (k < kmax && tid + k * NT < n) add(pmr[k]);
    } else {
      for (int i = tid; i < n; i += NT) add(pbar[i]);
    }
  }
  __syncthreads();
  unsigned long long W, Pthr;
  unsigned long long A = 0;   // mass of keys strictly above the threshold's bin / prefix range
  {
    // suffix sums from the top bin: thread k owns bins [4k, 4k + 4)
    constexpr int PER = FINE_BINS / NT;
    unsigned long long hb[PER], loc = 0;
#pragma unroll
    for (int b = 0; b < PER; ++b) {
      hb[b] = ((unsigned long long)sh.hist_hi[tid * PER + b] << 16) + sh.hist_lo[tid * PER + b];
      loc += hb[b];
    }
    unsigned long long suf = loc;   // inclusive suffix scan across the warp (higher lane = higher bins)
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      unsigned long long x = __shfl_down_sync(0xffffffffu, suf, o);
      if (lane + o < 32) suf += x;
    }
    if (lane == 0) sh.redu[w] = suf;
    __syncthreads();
    unsigned long long above = 0;
    W = 0;
    for (int x = 0; x < NW; ++x) {
      const unsigned long long r = sh.redu[x];
      W += r;
      if (x > w) above += r;
    }
    // hit  <=>  mass strictly before the entry  <  p * W
    Pthr = (unsigned long long)ceil((double)p.top_p * (double)W);
    unsigned long long sab = above + (suf - loc);   // mass above this thread's top bin
#pragma unroll
    for (int b = PER - 1; b >= 0; --b) {
      if (sab < Pthr && Pthr <= sab + hb[b]) {
        sh.star = tid * PER + b;
        sh.redu[NW] = sab;
      }
      sab += hb[b];
    }
    __syncthreads();
  }
  uint32_t theta = 0xffffffffu;
  int cnt_eq = 0;
  bool found_all = false;
  const int bstar = sh.star;
  if (bstar > 0 && bstar < FINE_BINS - 1) {   // inside the window: rank the bin's entries exactly
    A = sh.redu[NW];
    auto offer = [&](float pm) {
      const uint32_t key = __float_as_uint(pm);
      if (fbin(key) == bstar) {
        const int x = atomicAdd(&sh.ncand, 1);
        if (x < MAX_CAND) sh.cand[x] = key;
      }
    };
    if (EPT > 0) {
#pragma unroll
      for (int k = 0; k < R; ++k)
        if (k < kmax && tid + k * NT < n) offer(pmr[k]);
    } else {
      for (int i = tid; i < n; i += NT) offer(pbar[i]);
    }
    __syncthreads();
    const int c = sh.ncand;
    if (c <= MAX_CAND) {
      // candidate x carries the threshold iff  A + mass(keys above it) < Pthr <= that + mass(keys equal)
      if (tid < c) {
        const uint32_t mine = sh.cand[tid];
        const unsigned long long wm = mass_of(__uint_as_float(mine));
        unsigned long long gt = 0;
        int eqc = 0;
        for (int x = 0; x < c; ++x) {
          const uint32_t kx = sh.cand[x];
          if (kx > mine) gt += mass_of(__uint_as_float(kx));
          eqc += (kx == mine);
        }
        if (A + gt < Pthr && Pthr <= A + gt + (unsigned long long)eqc * wm) {
          sh.theta = mine;            // every carrier writes the same three values
          sh.A_theta = A + gt;
          sh.cnt_theta = eqc;
        }
      }
      __syncthreads();
      if (sh.cnt_theta > 0) {
        theta = sh.theta;
        A = sh.A_theta;
        cnt_eq = sh.cnt_theta;
        found_all = true;
      }
    }
  }
  if (!found_all) {
    // ---- general path: MSB-first radix passes over the fp32 bits of pbar, 8 bits each
    A = 0;
    uint32_t prefix = 0;
    found_all = true;
    for (int pass = 0; pass < 4; ++pass) {
      const int sft = 24 - 8 * pass;
      const int wid = 8;
      const int nb = 1 << wid;
      __syncthreads();
      for (int b = tid; b < nb; b += NT) { sh.hist_lo[b] = 0u; sh.hist_hi[b] = 0u; }
      if (tid == 0) sh.star = -1;
      __syncthreads();
      auto add = [&](float pm) {
        const uint32_t key = __float_as_uint(pm);
        const bool match = (pass == 0) || ((key >> (sft + wid)) == (prefix >> (sft + wid)));
        if (match) {
          const unsigned long long m = mass_of(pm);
          const int b = (key >> sft) & (nb - 1);
          atomicAdd(&sh.hist_lo[b], (unsigned)(m & 0xffffu));
          atomicAdd(&sh.hist_hi[b], (unsigned)(m >> 16));
        }
      };
      if (EPT > 0) {
#pragma unroll
        for (int k = 0; k < R; ++k)
          if (k < kmax && tid + k * NT < n) add(pmr[k]);
      } else {
        for (int i = tid; i < n; i += NT) add(pbar[i]);
      }
      __syncthreads();
      // suffix sums from the top bin: thread k owns bins [k*per, (k+1)*per)
      const int per = nb / NT;
      unsigned long long hb[HIST_BINS / NT];
      unsigned long long loc = 0;
#pragma unroll
      for (int b = 0; b < HIST_BINS / NT; ++b) {
        hb[b] = 0;
        if (b < per) hb[b] = ((unsigned long long)sh.hist_hi[tid * per + b] << 16) + sh.hist_lo[tid * per + b];
        loc += hb[b];
      }
      unsigned long long suf = loc;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        unsigned long long x = __shfl_down_sync(0xffffffffu, suf, o);
        if (lane + o < 32) suf += x;
      }
      if (lane == 0) sh.redu[w] = suf;
      __syncthreads();
      unsigned long long above = 0;
      for (int x = w + 1; x < NW; ++x) above += sh.redu[x];
      unsigned long long sab = A + above + (suf - loc);   // mass above this thread's top bin
#pragma unroll
      for (int b = HIST_BINS / NT - 1; b >= 0; --b) {
        if (b < per) {
          if (sab < Pthr && Pthr <= sab + hb[b]) {
            sh.star = tid * per + b;
            sh.redu[NW] = sab;
          }
          sab += hb[b];
        }
      }
      __syncthreads();
      const int dstar = sh.star;
      if (dstar < 0) { found_all = false; break; }
      prefix |= (uint32_t)dstar << sft;
      A = sh.redu[NW];
    }
    __syncthreads();
    if (!found_all) {
      if (tid == 0) atomicOr(st.errword, ERR_NUCLEUS);
      prefix = 0xffffffffu;  // nothing is a hit
    }
    // entries whose pbar equals the threshold key share one mass; the earliest positions win
    theta = prefix;
    int eq = 0;
    if (EPT > 0) {
#pragma unroll
      for (int k = 0; k < R; ++k)
        if (k < kmax && tid + k * NT < n) eq += (__float_as_uint(pmr[k]) == theta);
    } else {
      for (int i = tid; i < n; i += NT) eq += (__float_as_uint(pbar[i]) == theta);
    }
    eq = warp_sum_i(eq);
    if (lane == 0) sh.eq[w] = eq;
    __syncthreads();
    for (int x = 0; x < NW; ++x) cnt_eq += sh.eq[x];
  }
  if (EPT > 0 && cnt_eq > 1) {   // the rank among equal keys needs every entry's key: spill them
#pragma unroll
    for (int k = 0; k < R; ++k)
      if (k < kmax && tid + k * NT < n) pbar[tid + k * NT] = pmr[k];
    __syncthreads();
  }
  const unsigned long long w_theta = mass_of(__uint_as_float(theta));

  // ---- steps 2-3: CRF/tau update; step 4 candidates
  // step 4 runs once the head is evict_every entries over its budget, and then for all of them
  const int k_evict = (!p.hold && n - fr.budget >= p.evict_every) ? n - fr.budget : 0;
  uint32_t bk0 = 0xffffffffu, bk1 = 0xffffffffu, bk2 = 0xffffffffu;
  int bidx = -1, nhit = 0;
  auto update = [&](int i, float pm, int pos_i, int tau, float crf, float dec) {
    const uint32_t key = __float_as_uint(pm);
    bool hit = key > theta && found_all;
    if (key == theta && found_all) {
      unsigned long long rank = 0;
      if (cnt_eq > 1)
        for (int x = 0; x < n; ++x)
          rank += (__float_as_uint(pbar[x]) == theta) && (st.meta_pos[mb + x] < pos_i);
      hit = (A + rank * w_theta) < Pthr;
    }
    float ct = __fmul_rn(dec, crf);
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
  };
  if (EPT > 8) {   // many entries per thread: eight at a time, their stored state requested together
#pragma unroll
    for (int k0 = 0; k0 < R; k0 += 8) {
      if (k0 < kmax) {
        int pos4[8], tau4[8];
        float crf4[8], dec4[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const size_t i = mb + min(tid + (k0 + j) * NT, n - 1);
          pos4[j] = ld_i32(st.meta_pos + i);
          tau4[j] = ld_i32(st.meta_tau + i);
          crf4[j] = ld_f32(st.meta_crf + i);
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) dec4[j] = __ldg(st.tab + (p.t - min(tau4[j], p.t)));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const int i = tid + (k0 + j) * NT;
          if (k0 + j < R && i < n) update(i, pmr[k0 + j < R ? k0 + j : 0], pos4[j], tau4[j], crf4[j], dec4[j]);
        }
      }
    }
  } else if (EPT > 0) {
    float dec_r[R];
#pragma unroll
    for (int k = 0; k < R; ++k) dec_r[k] = __ldg(st.tab + (p.t - min(tau_r[k], p.t)));
#pragma unroll
    for (int k = 0; k < R; ++k) {
      const int i = tid + k * NT;
      if (i < n) update(i, pmr[k], pos_r[k], tau_r[k], crf_r[k], dec_r[k]);
    }
  } else {
    for (int i = tid; i < n; i += NT) {
      const int tau = st.meta_tau[mb + i];
      update(i, pbar[i], st.meta_pos[mb + i], tau, st.meta_crf[mb + i], st.tab[p.t - tau]);
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
    if (lane == 0) { sh.amin[w * 4] = (int)bk0; sh.amin[w * 4 + 1] = (int)bk1; sh.amin[w * 4 + 2] = (int)bk2; sh.amin[w * 4 + 3] = bidx; }
    __syncthreads();
    if (tid == 0) {
      uint32_t a0 = (uint32_t)sh.amin[0], a1 = (uint32_t)sh.amin[1], a2 = (uint32_t)sh.amin[2];
      int ai = sh.amin[3];
      for (int x = 1; x < NW; ++x) {
        const uint32_t o0 = (uint32_t)sh.amin[x * 4], o1 = (uint32_t)sh.amin[x * 4 + 1], o2 = (uint32_t)sh.amin[x * 4 + 2];
        const bool less = (o0 != a0) ? (o0 < a0) : ((o1 != a1) ? (o1 < a1) : (o2 < a2));
        if (less) { a0 = o0; a1 = o1; a2 = o2; ai = sh.amin[x * 4 + 3]; }
      }
      // the leaving entry's place is where the next arriving token is written
      st.hole[uid] = ai;
      st.n_cur[uid] = n - 1;
      atomicAdd(&st.counters[2], 1ull);
    }
    n_after = n - 1;
  } else if (k_evict > 1) {
    __syncthreads();
    if (p.append && k_evict > p.evict_every && tid == 0) atomicOr(st.errword, ERR_OVER_EVICT);
    evict_many(st, uid, seq, n, min(k_evict, n - 1), p.t, p.release != 0, sh.ev, reinterpret_cast<int*>(pbar),
               p.rows_absent == 0);
    n_after = n - min(k_evict, n - 1);
  }
  if (n_after == n && tid == 0 && !p.hold) keep_all(st, uid, seq, n, p.append != 0);
  return n_after;   // the head's length after the step
}

template <int G>
__global__ void __launch_bounds__(NT, 5) lrfu_kernel(const DecodeParams p) {
  __shared__ LrfuSmem sh;
  const State& st = p.st;
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + p.layer) * st.H + head;
  // one batch of requests: the length, the budget, the softmax reference, and the logit rows the
  // common path needs (requested for a full thread's worth, clamped to the scratch)
  int n_raw = ld_i32(st.n_cur + uid);
  const int g_plan = (threadIdx.x == 0 && p.plan_append >= 0) ? ld_i32(p.plan.gplan + u) : 0;   // used at the very end
  if (p.n_limit > 0) n_raw = min(n_raw, p.n_limit);
  const int n = n_raw + p.append;
  int n_new = n;   // the head's length after this launch
  if (p.track) {
    Front<G> fr;
    fr.budget = ld_i32(st.budget + uid);
#pragma unroll
    for (int g = 0; g < G; ++g) {
      fr.m[g] = ld_f32(p.sc.mfin + u * (2 * QH) + g);
      fr.l[g] = ld_f32(p.sc.mfin + u * (2 * QH) + QH + g);
    }
    {
      const float* S = p.sc.logits + (size_t)u * p.sc.cap_s * QH;
#pragma unroll
      for (int k = 0; k < FRONT; ++k) {
        const int i = min((int)threadIdx.x + k * NT, p.sc.cap_s - 1);
        fr.ra[k] = ld_f32x4(S + (size_t)i * QH);
        fr.rb[k] = (G > 4) ? ld_f32x4(S + (size_t)i * QH + 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (n <= 0) {
      if (threadIdx.x == 0 && !p.hold) { st.n_cur[uid] = 0; st.hole[uid] = 0; }
      n_new = 0;
    } else if (p.literal && n < fr.budget) {   // Algorithm 1's first line as printed: nothing runs below the budget
      if (threadIdx.x == 0 && !p.hold) keep_all(st, uid, seq, n, p.append != 0);
    } else if (n <= FRONT * NT) {
      n_new = lrfu_unit<G, FRONT>(p, u, uid, seq, n, sh, fr);
    } else if (n <= 10 * NT) {
      n_new = lrfu_unit<G, 10>(p, u, uid, seq, n, sh, fr);
    } else if (n <= 17 * NT) {
      n_new = lrfu_unit<G, 17>(p, u, uid, seq, n, sh, fr);
    } else {
      n_new = lrfu_unit<G, 0>(p, u, uid, seq, n, sh, fr);
    }
  } else if (threadIdx.x == 0) {
    keep_all(st, uid, seq, n, p.append != 0);   // no Algorithm 1: the head keeps its new entry
  }
  if (threadIdx.x == 0) atomicAdd(&st.counters[0], (unsigned long long)max(n, 0));
  if (p.plan_append < 0) return;
  // ---- The layer's plan names pieces by (head, j of k), so it stays correct while heads grow or
  // shrink a little; a head whose group count has drifted from the planned one by an eighth (at
  // least two), or a next launch of another kind than this one, marks it stale, and the CTA that
  // finishes last (it then knows every head's new length) writes a new one.  In steady state (one
  // entry arrives, one leaves) nothing is written.  Thread 0 wrote the head's new length itself,
  // so the release of its count makes that length visible to whoever acquires the last count.
  if (threadIdx.x == 0) {
    const int g_new = (n_new + p.plan_append + GRP - 1) / GRP;
    if (abs(g_new - g_plan) >= max(2, g_plan >> 3) || p.append != p.plan_append) atomicOr(p.done_ctr + 1, 1);
    int done;
    asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(done) : "l"(p.done_ctr) : "memory");
    int last = (done == (int)gridDim.x - 1);
    if (last) {
      *p.done_ctr = 0;
      last = atomicExch(p.done_ctr + 1, 0);   // stale?
    }
    sh.is_last = last;
  }
  __syncthreads();
  if (!sh.is_last) return;
  write_plan(st, p.plan, p.layer, p.plan_append, 0, p.plan_warps, p.plan_grid, reinterpret_cast<int*>(&sh), sh.ev);
}

}  // namespace ckv
