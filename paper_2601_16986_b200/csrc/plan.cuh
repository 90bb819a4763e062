// Launch plan of a layer's attention kernel: which warp streams which groups of which head.
//
// Every head is cut into pieces of nearly equal length, at most T groups (pages of 16 keys)
// each, with T the smallest bound for which the pieces of all heads fit the grid's warps: one
// piece per warp, no warp with more than T groups, whatever the heads' lengths are (after the
// budgets have been reallocated heads hold a few hundred to a few thousand entries).  Pieces go
// round the SMs one by one, so every SM streams the same number of them to within one.  With
// more heads than warps every head is one piece and a warp takes several in turn.  A head of
// several pieces is merged from their partial results.  The plan only depends on the heads'
// lengths, so it is written by whichever kernel changed them (the LRFU kernel of the layer's
// previous step once a head has drifted from the planned length, the shrink pass of a
// reallocation, the prompt insertion) and the attention kernel starts streaming without deriving
// anything but its pieces' bounds from the heads' current lengths.
#pragma once
#include "common.cuh"

namespace ckv {

// Called by all NT threads of one CTA.  `gs` is shared memory for U + 1 ints, `red` for NW + 1.
// append: the plan is for a decode step (every head one entry longer than now); n_limit > 0: for
// a scoring pass over the first n_limit entries of every head.
__device__ __forceinline__ void write_plan(const State& st, const Plan& pl, int layer, int append, int n_limit, int nWarps,
                                        int grid, int* gs, int* red) {
  const int U = st.batch * st.H, tid = threadIdx.x;
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
  if ((tid & 31) == 0) red[tid >> 5] = gmax;
  __syncthreads();
  for (int x = 0; x < NW; ++x) gmax = max(gmax, red[x]);
  empty = __syncthreads_or(empty);
  if (empty) {   // a head without entries cannot be attended: nothing is planned
    if (tid == 0) atomicOr(st.errword, ERR_PLAN);
    Gtot = 0;
  }
  // ---- the piece bound T: the smallest for which sum ceil(g_u / T) <= nWarps (none when there
  // are more heads than warps: one piece per head then)
  int T = 0x7fffffff;
  if (Gtot > 0 && U <= nWarps) {
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
    T = max(lo, min(GMIN, gmax));   // pieces shorter than GMIN groups cost more in starts and merges than they gain
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
      for (int j = 0; j < k; ++j) pl.desc[start + j] = make_int4(u, j, k, 0);
    }
  }
  // ---- which warp takes which pieces: consecutive pieces go to consecutive warps, so that most
  // heads have all their pieces in one CTA and are merged in its shared memory (with fewer pieces
  // than warps the last CTAs stay idle); with more pieces than warps every warp takes a run of
  // consecutive pieces
  const int per = (pieces + nWarps - 1) / max(nWarps, 1);
  for (int pw = tid; pw < nWarps; pw += NT) {
    int2 r = make_int2(0, 0);
    if (pieces <= nWarps) {
      if (pw < pieces) r = make_int2(pw, pw + 1);
    } else {
      const int i0 = min(pieces, pw * per);
      r = make_int2(i0, min(pieces, i0 + per));
    }
    pl.wrange[pw] = r;
  }
  if (tid == 0) {
    pl.hdr[0] = pieces;
    pl.hdr[1] = Gtot;
    pl.hdr[2] = nWarps;
    pl.hdr[3] = append;
  }
}

// The plan as a kernel of its own: one CTA per layer of `layers` consecutive layers starting at
// layer0 (after a prompt insertion, a reallocation, or any edit of a head's state from the host).
__global__ void __launch_bounds__(NT) plan_kernel(State st, const Plan* plans, int layer0, int append, int n_limit,
                                                  int nWarps, int grid) {
  __shared__ int s_gs[MAX_UNITS_PER_CALL + 1];
  __shared__ int s_red[NW + 1];
  write_plan(st, plans[layer0 + blockIdx.x], layer0 + blockIdx.x, append, n_limit, nWarps, grid, s_gs, s_red);
}

}  // namespace ckv
