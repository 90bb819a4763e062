// Launch plan of a layer's attention kernel: which warp streams which groups of which head.
//
// Every head is cut into k = ceil(g / T) pieces of nearly equal length, at most T groups (pages of
// 16 keys) each, one piece per warp, and all pieces of a head are placed in consecutive warps of
// ONE CTA, where the head is merged in shared memory (a head of more than eight pieces takes whole
// CTAs and one shorter run).  T is the smallest bound for which such a placement fits the grid,
// whatever the heads' lengths are (after the budgets have been reallocated heads hold a few hundred
// to a few thousand entries); longer pieces are taken where they keep heads inside one CTA at less
// cost than the merge through global memory they avoid.  With more heads than warps every head is
// one piece and a warp takes several in turn.  The plan only depends on the heads' lengths, so it
// is written by whichever kernel changed them (the LRFU kernel of the layer's previous step once a
// head has drifted from the planned length, the shrink pass of a reallocation, the prompt
// insertion) and the attention kernel starts streaming without deriving anything but its pieces'
// bounds from the heads' current lengths.
#pragma once
#include "common.cuh"

namespace ckv {

// CTAs a set of heads needs when the pieces of a head have to sit in consecutive warps of one CTA:
// `full` CTAs are taken whole (eight pieces of a head with eight or more), cnt[s] runs of s < 8
// pieces are packed best fit, longest first.  A run goes to the open CTA with the fewest free
// warps that still holds it, so a CTA with c free warps takes c / s runs of length s one after the
// other: the loop below moves whole classes of CTAs at once and counts exactly what the
// run-by-run placement in write_plan() does.
__host__ __device__ __forceinline__ int ctas_needed(int full, const int (&cnt)[8]) {
  int open[9] = {0, 0, 0, 0, 0, 0, 0, 0, 0};   // open[c]: CTAs with c free warps
  int ctas = full;
#pragma unroll
  for (int s = 7; s >= 1; --s) {
    int n = cnt[s];
#pragma unroll
    for (int c = s; c <= 8; ++c) {
      const int q = c / s;                              // runs one such CTA takes
      const int have = (c == 8) ? (n + q - 1) / q : open[c];   // fresh CTAs are not counted in open[]
      const int nb = have < n / q ? have : n / q;       // CTAs filled with q runs
      int left = c - q * s;
      if (c == 8) ctas += nb; else open[c] -= nb;
      open[left] += nb;
      n -= nb * q;
      if (n > 0 && n < q && have > nb) {                // one more takes the rest
        if (c == 8) ++ctas; else --open[c];
#pragma unroll
        for (int nn = 1; nn < 8; ++nn)
          if (nn < q && n == nn) open[c - nn * s] += 1;
        n = 0;
      }
    }
  }
  return ctas;
}

// Called by all NT threads of one CTA.  `gs` is shared memory for U + 1 ints, `red` for 320.
// append: the plan is for a decode step (every head one entry longer than now); n_limit > 0: for
// a scoring pass over the first n_limit entries of every head.
__device__ __forceinline__ void write_plan(const State& st, const Plan& pl, int layer, int append, int n_limit, int nWarps,
                                        int grid, int* gs, int* red) {
  const int U = st.batch * st.H, tid = threadIdx.x, lane = tid & 31;
  // ---- groups per head
  int mine = 0, gmax = 0, empty = 0;
  for (int u = tid; u < U; u += NT) {
    const int uid = ((u / st.H) * st.L + layer) * st.H + (u % st.H);
    int n = __ldcg(st.n_cur + uid);   // (other CTAs of the calling kernel may just have written it: not from L1)
    if (n_limit > 0) n = min(n, n_limit);
    const int g = (n + append + GRP - 1) / GRP;
    gs[u] = g;
    mine += g;
    gmax = max(gmax, g);
    empty |= (g == 0);
  }
  int Gtot;
  block_excl_scan(mine, red, Gtot);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) gmax = max(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
  __syncthreads();
  if (lane == 0) red[tid >> 5] = gmax;
  __syncthreads();
  for (int x = 0; x < NW; ++x) gmax = max(gmax, red[x]);
  empty = __syncthreads_or(empty);
  if (empty) {   // a head without entries cannot be attended: nothing is planned
    if (tid == 0) atomicOr(st.errword, ERR_PLAN);
    Gtot = 0;
  }
  // ---- the piece bound T.  Heads are cut into ceil(g_u / T) pieces; the smallest T is wanted for
  // which all heads can be placed with every head's pieces inside one CTA (such a head is merged in
  // shared memory; one that straddles CTAs goes through global memory and a ticket, which costs the
  // launch several microseconds at its end).  32 candidates are tried at once: warp x counts the
  // runs of every length over the heads u = x mod 8, lane c for T0 + c; warp 0 then packs them.
  int T = 0x7fffffff;
  bool packed = false;
  int* hist = red + 16;   // [32][4]: counts of two run lengths per word, 16 bits each (U < 65536)
  if (Gtot > 0 && U <= nWarps && grid * NW == nWarps && grid <= 256 && nWarps < 4096) {
    // A launch with few groups per warp is bound by the steps a head's result goes through, not by
    // bytes: pieces are then made long enough (up to GLAT groups) for the longest head to stay inside
    // one CTA, whose merge is one barrier instead of a trip through global memory.
    const int gfloor = min(gmax, max(GMIN, min(GLAT, (gmax + NW - 1) / NW)));
    const int T0 = max(max(1, (Gtot + nWarps - 1) / nWarps), gfloor);   // pieces shorter than GMIN groups
                                                                                // cost more in starts and merges than they gain
    // first feasible bound among Tfirst .. Tfirst + 31, or -1
    auto first_that_packs = [&](int Tfirst) {
      const int Tc = Tfirst + lane;
      if (tid < 128) hist[tid] = 0;
      __syncthreads();
      unsigned h4[4] = {0u, 0u, 0u, 0u};
      for (int u = tid >> 5; u < U; u += NW) {
        const int k = (gs[u] + Tc - 1) / Tc;
        const int r = k & 7;   // 0: nothing beyond whole CTAs
#pragma unroll
        for (int x = 0; x < 4; ++x) h4[x] += ((x > 0 && r == 2 * x) ? 1u : 0u) + ((r == 2 * x + 1) ? 0x10000u : 0u);
        h4[0] += (unsigned)(k >> 3);   // the low half of word 0 counts whole CTAs (there is no run of length 0)
      }
#pragma unroll
      for (int x = 0; x < 4; ++x) atomicAdd(reinterpret_cast<unsigned*>(hist) + lane * 4 + x, h4[x]);
      __syncthreads();
      if (tid < 32) {
        int cnt[8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const unsigned v = (unsigned)hist[lane * 4 + x];
          cnt[2 * x] = (int)(v & 0xffffu);
          cnt[2 * x + 1] = (int)(v >> 16);
        }
        const int full = cnt[0];
        const int ok = ctas_needed(full, cnt) <= grid;
        const unsigned m = __ballot_sync(0xffffffffu, ok);
        if (lane == 0) red[0] = m ? Tfirst + (__ffs(m) - 1) : -1;
      }
      __syncthreads();
      const int found = red[0];
      __syncthreads();
      return found;
    };
    for (int round = 0; round < 4 && !packed; ++round) {
      const int found = first_that_packs(T0 + round * 32);
      if (found > 0) { T = found; packed = true; }
    }
    // Heads of more than eight pieces go through global memory, which costs the end of the launch
    // about as much as seven groups of streaming.  When pieces long enough for the longest head to fit
    // one CTA (gmax / 8 groups) cost less than that -- streaming is bound by the longer of a warp's own
    // groups and its share of the HBM rate, 7/4 group times per group at full occupancy -- they are taken.
    const int Tb = (gmax + NW - 1) / NW;
    if (packed && Tb > T) {
      const int hbm = (int)(((long long)Gtot * 7 / 4 + nWarps - 1) / nWarps);
      if (Tb <= max(T, hbm) + 7) {
        const int found = first_that_packs(Tb);
        if (found > 0 && found <= Tb + 2) T = found;
      }
    }
  }
  if (!packed && Gtot > 0 && U <= nWarps) {
    // fallback: the smallest T for which sum ceil(g_u / T) <= nWarps, heads laid over the warps end to end
    int lo = max(1, (Gtot + nWarps - 1) / nWarps), hi = max(lo, gmax);   // feasible at hi: one piece per head
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      int cnt = 0;
      for (int u = tid; u < U; u += NT) cnt += (gs[u] + mid - 1) / mid;
      int tot;
      block_excl_scan(cnt, red, tot);
      __syncthreads();
      if (tot <= nWarps) hi = mid; else lo = mid + 1;
    }
    T = max(lo, min(GMIN, gmax));
  }
  // ---- pieces per head, their prefix sums, the descriptors
  int pieces = 0;
  for (int b0 = 0; b0 < U; b0 += NT) {
    const int u = b0 + tid;
    const int g = (u < U && Gtot > 0) ? gs[u] : 0;
    const int k = g == 0 ? 0 : (T == 0x7fffffff ? 1 : (g + T - 1) / T);
    int tot;
    const int start = pieces + block_excl_scan(k, red, tot);
    pieces += tot;
    if (u < U) {
      pl.npc[u] = k;
      pl.gplan[u] = g;
      // the last word: 1 when the head's k pieces sit in consecutive warps of one CTA, each warp with
      // nothing else to stream; 2 when they sit that way in runs of eight (whole CTAs) and one shorter run
      const int together = k <= 1 ? 0 : (packed ? (k <= NW ? 1 : 2) : ((start & (NW - 1)) + k <= NW ? 1 : 0));
      for (int j = 0; j < k; ++j) pl.desc[start + j] = make_int4(u, j, k, together);
      if (packed) gs[u] = (start << 12) | k;
    }
  }
  if (packed) {
    for (int pw = tid; pw < nWarps; pw += NT) pl.wrange[pw] = make_int4(0, 0, -1, 0);
    __syncthreads();
    if (tid < 32) {
      // every lane keeps the same books; the lanes share the stores
      int* nxt = red + 16;   // [grid] next CTA in the list of its class
      int next_cta = 0, over = 0;
      for (int b0 = 0; b0 < U && !over; b0 += 32) {   // whole CTAs first
        const int v = (b0 + lane < U) ? gs[b0 + lane] : 0;
        unsigned m = __ballot_sync(0xffffffffu, (v & 4095) >= NW);
        while (m) {
          const int b = __ffs(m) - 1;
          m &= m - 1;
          const int vv = __shfl_sync(0xffffffffu, v, b);
          const int start = vv >> 12, kk = vv & 4095, nw = (kk >> 3) * NW;
          if (next_cta * NW + nw > nWarps) { over = 1; break; }
          for (int x = lane; x < nw; x += 32)
            pl.wrange[next_cta * NW + x] = make_int4(start + x, start + x + 1, b0 + b, x | (kk << 12) | ((kk <= NW ? 1 : 2) << 24));
          next_cta += nw / NW;
        }
      }
      int head[8] = {-1, -1, -1, -1, -1, -1, -1, -1};   // head[c]: first of the CTAs with c free warps
#pragma unroll
      for (int s = 7; s >= 1; --s) {
        for (int b0 = 0; b0 < U && !over; b0 += 32) {
          const int v = (b0 + lane < U) ? gs[b0 + lane] : 0;
          unsigned m = __ballot_sync(0xffffffffu, (v & 7) == s);
          while (m) {
            const int b = __ffs(m) - 1;
            m &= m - 1;
            const int vv = __shfl_sync(0xffffffffu, v, b);
            const int start = vv >> 12, k = vv & 4095;
            int cta = -1, c = 8;
#pragma unroll
            for (int cc = s; cc <= 7; ++cc)
              if (cta < 0 && head[cc] >= 0) {
                cta = head[cc];
                head[cc] = nxt[cta];
                c = cc;
              }
            if (cta < 0) {
              if (next_cta >= grid) { over = 1; break; }
              cta = next_cta++;
            }
            const int left = c - s;
#pragma unroll
            for (int dd = 1; dd <= 7; ++dd)
              if (left == dd) {
                nxt[cta] = head[dd];
                head[dd] = cta;
              }
            __syncwarp();
            const int j0 = k - s;   // the pieces before these took whole CTAs
            if (lane < s)
              pl.wrange[cta * NW + (NW - c) + lane] = make_int4(start + j0 + lane, start + j0 + lane + 1, b0 + b,
                                                                (j0 + lane) | (k << 12) | ((k <= 1 ? 0 : (k <= NW ? 1 : 2)) << 24));
          }
        }
      }
      if (over && lane == 0) {   // cannot happen while ctas_needed() counts what this loop does; never leave half a plan
        atomicOr(st.errword, ERR_PLAN);
        nWarps = -1;
      }
      nWarps = __shfl_sync(0xffffffffu, nWarps, 0);
    }
  } else {
    // heads end to end: consecutive pieces go to consecutive warps; with more pieces than warps
    // every warp takes a run of consecutive pieces
    const int per = (pieces + nWarps - 1) / max(nWarps, 1);
    for (int pw = tid; pw < nWarps; pw += NT) {
      int4 r = make_int4(0, 0, -1, 0);
      if (pieces <= nWarps) {
        if (pw < pieces) r = make_int4(pw, pw + 1, -1, 0);
      } else {
        const int i0 = min(pieces, pw * per);
        r = make_int4(i0, min(pieces, i0 + per), -1, 0);
      }
      pl.wrange[pw] = r;
    }
  }
  if (tid == 0) {
    pl.hdr[0] = pieces;
    pl.hdr[1] = Gtot;
    pl.hdr[2] = nWarps;   // (-1 after a failed placement: no launch accepts the plan)
    pl.hdr[3] = append;
  }
}

// The plan as a kernel of its own: one CTA per layer of `layers` consecutive layers starting at
// layer0 (after a prompt insertion, a reallocation, or any edit of a head's state from the host).
__global__ void __launch_bounds__(NT) plan_kernel(State st, const Plan* plans, int layer0, int append, int n_limit,
                                                  int nWarps, int grid) {
  __shared__ int s_gs[MAX_UNITS_PER_CALL + 1];
  __shared__ int s_red[320];
  write_plan(st, plans[layer0 + blockIdx.x], layer0 + blockIdx.x, append, n_limit, nWarps, grid, s_gs, s_red);
}

}  // namespace ckv
