// Set-up and periodic kernels around the decode step: prompt insertion, Algorithm 2
// (adaptive budget allocation) and the shrink pass that moves slot ownership between heads.
#pragma once
#include "common.cuh"
#include "evict.cuh"

namespace ckv {

// ---------------------------------------------------------------------------------------
// Prompt insertion for one layer: one CTA per (sequence, kv head).  Takes the pages that back
// list positions 0 .. P (the P entries and the place of the next arrival) from the sequence's
// free list, writes the K/V rows into them in the page layout and sets pos = i, CRF = 0 and
// tau = P - 1 (the time of the scoring pass that follows) or, when the prompt's last tokens
// are replayed one by one, tau = i (the token's own arrival time).
//   k, v: [batch][P][H][128] bf16
__global__ void __launch_bounds__(NT) prefill_insert_kernel(State st, int layer, const __nv_bfloat16* k,
                                                            const __nv_bfloat16* v, int P, int tau_is_pos) {
  __shared__ int s_top;
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + layer) * st.H + head;
  const size_t mb = (size_t)uid * st.cap;
  const int tid = threadIdx.x;
  const int need = P / GRP + 1;
  if (tid == 0) {
    int top = -1;
    if (P + 1 > st.cap) {
      atomicOr(st.errword, ERR_CAPACITY);
    } else {
      top = atomicSub(&st.free_top[seq], need);
      if (top < need) {
        atomicAdd(&st.free_top[seq], need);
        atomicOr(st.errword, ERR_FREE_UNDERFLOW);
        top = -1;
      }
    }
    s_top = top;
  }
  __syncthreads();
  const int top = s_top;
  if (top < 0) {
    if (tid == 0) { st.n_cur[uid] = 0; st.hole[uid] = 0; }
    return;
  }
  const int* stack = st.free_stack + (size_t)seq * st.pages_per_seq;
  int* pt = st.ptab + (size_t)uid * st.capg;
  for (int j = tid; j < need; j += NT) pt[j] = stack[top - 1 - j];
  for (int i = tid; i < P; i += NT) {
    st.meta_pos[mb + i] = i;
    st.meta_tau[mb + i] = tau_is_pos ? i : P - 1;
    st.meta_crf[mb + i] = 0.0f;
  }
  unsigned char* poolseq = st.pool + (size_t)seq * st.pages_per_seq * PAGE_BYTES;
  const int c = tid & 31;   // chunk of the entry's 512 bytes: K row, then V row
  for (int i = tid >> 5; i < P; i += NW) {
    const int page = stack[top - 1 - (i >> 4)];
    const size_t off = (((size_t)seq * P + i) * st.H + head) * HD * 2;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(c < 16 ? k : v) + off + (c & 15) * 16;
    *reinterpret_cast<uint4*>(poolseq + (size_t)page * PAGE_BYTES + chunk_offset(i & (GRP - 1), c)) =
        *reinterpret_cast<const uint4*>(src);
  }
  if (tid == 0) { st.n_cur[uid] = P; st.hole[uid] = P; st.npages[uid] = need; }
}

// ---------------------------------------------------------------------------------------
// A prompt longer than its heads' budgets is scored before it is stored: Algorithm 1 needs the
// scores of all P tokens but only the B survivors' rows ever need a place in the pool.
// Step 1 of three (one CTA per head): the P entries as metadata only (pos = i, CRF 0,
// tau = P - 1), the scaled logits of the last query's G heads against the prompt's keys, read
// from the caller's tensors, and the softmax reference point and normaliser per query head, all
// where the LRFU kernel expects them.
//   k: [batch][P][H][128]   q_last: [batch][Hq][128]
__global__ void __launch_bounds__(NT) prefill_score_kernel(State st, Scratch sc, int layer, const __nv_bfloat16* k,
                                                           const __nv_bfloat16* q_last, int P, int G, float scale,
                                                           float scale_log2) {
  __shared__ float s_q[QH * HD];
  __shared__ float s_red[NW][QH];
  __shared__ float s_m[QH];
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + layer) * st.H + head;
  const size_t mb = (size_t)uid * st.cap;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  if (P + 1 > st.cap) {
    if (tid == 0) { atomicOr(st.errword, ERR_CAPACITY); st.n_cur[uid] = 0; st.hole[uid] = 0; }
    return;
  }
  for (int x = tid; x < QH * HD; x += NT)
    s_q[x] = (x / HD < G) ? __bfloat162float(q_last[((size_t)u * G + x / HD) * HD + (x % HD)]) : 0.f;
  __syncthreads();
  float* S = sc.logits + (size_t)u * sc.cap_s * QH;
  float mx[QH];
#pragma unroll
  for (int g = 0; g < QH; ++g) mx[g] = -INFINITY;
  for (int i = tid; i < P; i += NT) {
    st.meta_pos[mb + i] = i;
    st.meta_tau[mb + i] = P - 1;
    st.meta_crf[mb + i] = 0.0f;
    const uint4* row = reinterpret_cast<const uint4*>(k + (((size_t)seq * P + i) * st.H + head) * HD);
    float acc[QH];
#pragma unroll
    for (int g = 0; g < QH; ++g) acc[g] = 0.f;
    for (int c = 0; c < HD / 8; ++c) {
      const uint4 v = row[c];
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
      float kv[8];
#pragma unroll
      for (int x = 0; x < 4; ++x) { const float2 f = __bfloat1622float2(h2[x]); kv[2 * x] = f.x; kv[2 * x + 1] = f.y; }
#pragma unroll
      for (int g = 0; g < QH; ++g)
#pragma unroll
        for (int x = 0; x < 8; ++x) acc[g] = fmaf(s_q[g * HD + c * 8 + x], kv[x], acc[g]);
    }
    float out[QH];
#pragma unroll
    for (int g = 0; g < QH; ++g) {
      out[g] = __fmul_rn(acc[g], scale);
      mx[g] = fmaxf(mx[g], acc[g] * scale_log2);
    }
    *reinterpret_cast<float4*>(S + (size_t)i * QH) = make_float4(out[0], out[1], out[2], out[3]);
    *reinterpret_cast<float4*>(S + (size_t)i * QH + 4) = make_float4(out[4], out[5], out[6], out[7]);
  }
#pragma unroll
  for (int g = 0; g < QH; ++g) {
    const float m = warp_max(mx[g]);
    if (lane == 0) s_red[w][g] = m;
  }
  __syncthreads();
  if (tid < QH) {
    float m = s_red[0][tid];
    for (int x = 1; x < NW; ++x) m = fmaxf(m, s_red[x][tid]);
    s_m[tid] = m;
  }
  __syncthreads();
  float sum[QH];
#pragma unroll
  for (int g = 0; g < QH; ++g) sum[g] = 0.f;
  const float to_log2 = scale_log2 / scale;
  for (int i = tid; i < P; i += NT) {
#pragma unroll
    for (int g = 0; g < QH; ++g) sum[g] += ex2(S[(size_t)i * QH + g] * to_log2 - s_m[g]);
  }
  __syncthreads();
#pragma unroll
  for (int g = 0; g < QH; ++g) {
    const float x = warp_sum(sum[g]);
    if (lane == 0) s_red[w][g] = x;
  }
  __syncthreads();
  if (tid < G) {
    float l = 0.f;
    for (int x = 0; x < NW; ++x) l += s_red[x][tid];
    sc.mfin[u * (2 * QH) + tid] = s_m[tid];
    sc.mfin[u * (2 * QH) + QH + tid] = l;
  }
  if (tid == 0) { st.n_cur[uid] = P; st.hole[uid] = P; st.npages[uid] = 0; }
}

// Step 3 (step 2 is the LRFU kernel, which leaves the survivors' metadata dense): the pages that
// back the survivors and the place of the next arrival are taken from the free list and the
// survivors' rows are fetched from the prompt tensors by their token positions.
__global__ void __launch_bounds__(NT) prefill_rows_kernel(State st, int layer, const __nv_bfloat16* k,
                                                          const __nv_bfloat16* v, int P) {
  __shared__ int s_top;
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + layer) * st.H + head;
  const size_t mb = (size_t)uid * st.cap;
  const int tid = threadIdx.x;
  const int n = st.n_cur[uid];
  const int need = n / GRP + 1;
  if (tid == 0) {
    int top = atomicSub(&st.free_top[seq], need);
    if (top < need) {
      atomicAdd(&st.free_top[seq], need);
      atomicOr(st.errword, ERR_FREE_UNDERFLOW);
      top = -1;
    }
    s_top = top;
  }
  __syncthreads();
  const int top = s_top;
  if (top < 0) {
    if (tid == 0) { st.n_cur[uid] = 0; st.hole[uid] = 0; }
    return;
  }
  const int* stack = st.free_stack + (size_t)seq * st.pages_per_seq;
  int* pt = st.ptab + (size_t)uid * st.capg;
  for (int j = tid; j < need; j += NT) pt[j] = stack[top - 1 - j];
  unsigned char* poolseq = st.pool + (size_t)seq * st.pages_per_seq * PAGE_BYTES;
  const int c = tid & 31;
  for (int i = tid >> 5; i < n; i += NW) {
    const int page = stack[top - 1 - (i >> 4)];
    const int tok = min(max(st.meta_pos[mb + i], 0), P - 1);
    const size_t off = (((size_t)seq * P + tok) * st.H + head) * HD * 2;
    const unsigned char* src = reinterpret_cast<const unsigned char*>(c < 16 ? k : v) + off + (c & 15) * 16;
    *reinterpret_cast<uint4*>(poolseq + (size_t)page * PAGE_BYTES + chunk_offset(i & (GRP - 1), c)) =
        *reinterpret_cast<const uint4*>(src);
  }
  if (tid == 0) st.npages[uid] = need;
}

// ---------------------------------------------------------------------------------------
// Brings one step's q, k_new and v_new from page-locked host memory (read over the bus through
// its device mapping, 16 bytes per thread) into the staging buffers: one launch instead of three
// copies.  It runs in the caller's stream directly ahead of the step's attention kernel, both
// launched with programmatic stream serialisation: this kernel lets the attention kernel start
// at once, fetches while the attention kernel of the previous layer is still running, and only
// then waits for that kernel, so that its own completion, which the attention kernel behind it
// waits for, implies the completion of everything ahead.
__global__ void __launch_bounds__(NT) stage_in_kernel(uint4* __restrict__ dq, uint4* __restrict__ dk,
                                                      uint4* __restrict__ dv, const uint4* __restrict__ hq,
                                                      const uint4* __restrict__ hk, const uint4* __restrict__ hv,
                                                      int nq, int nk) {
  asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory");
  const int i = blockIdx.x * NT + threadIdx.x;
  if (i < nq) dq[i] = hq[i];
  else if (i < nq + nk) dk[i - nq] = hk[i - nq];
  else if (i < nq + 2 * nk) dv[i - nq - nk] = hv[i - nq - nk];
  asm volatile("griddepcontrol.wait;\n" ::: "memory");
}

// ---------------------------------------------------------------------------------------
// Algorithm 2 input: per head, the sum of CRF decayed to t_last over the retained entries,
// each term truncated to 2^-32 fixed point so the sum does not depend on the order.
__global__ void __launch_bounds__(NT) crf_sum_kernel(State st, int t_last, long long* Asum) {
  __shared__ long long s_red[NW];
  const int uid = blockIdx.x;
  const size_t mb = (size_t)uid * st.cap;
  const int n = st.n_cur[uid], hole = st.hole[uid];
  long long acc = 0;
  for (int x = threadIdx.x; x < n; x += NT) {
    const int i = live_pos(x, hole);
    const float d = __fmul_rn(st.tab[t_last - st.meta_tau[mb + i]], st.meta_crf[mb + i]);
    acc += (long long)((double)d * 4294967296.0);
  }
  acc = (long long)warp_sum_u64((unsigned long long)acc);
  if ((threadIdx.x & 31) == 0) s_red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    long long tot = 0;
    for (int x = 0; x < NW; ++x) tot += s_red[x];
    Asum[uid] = tot;
  }
}

// Block-wide: hand `extra` whole slots to the m heads listed in who[] in proportion to x[]:
// floor of the real share, then one more each by largest fractional part (ties to the
// lower head index).  Every fp64 operation is a single correctly rounded one, in the
// order a sequential evaluation of the same formulas takes them.
__device__ void share_out(long long extra, const int* who, int m, const double* x, long long* add,
                          double* frac, int* order, double* s_d, long long* s_ll) {
  const int tid = threadIdx.x;
  if (m <= 0 || extra <= 0) return;
  if (tid == 0) {
    double W = 0.0;
    for (int j = 0; j < m; ++j) W = __dadd_rn(W, x[who[j]]);
    s_d[0] = W;
  }
  __syncthreads();
  const double W = s_d[0];
  long long given = 0;
  for (int j = tid; j < m; j += NT) {
    const int k = who[j];
    const double xs = (W > 0.0) ? __ddiv_rn(__dmul_rn((double)extra, x[k]), W)
                                : __ddiv_rn((double)extra, (double)m);
    const double f = floor(xs);
    add[k] += (long long)f;
    given += (long long)f;
    frac[j] = __dsub_rn(xs, f);
  }
  given = (long long)warp_sum_u64((unsigned long long)given);
  if ((tid & 31) == 0) s_ll[tid >> 5] = given;
  __syncthreads();
  long long left = extra;
  for (int w = 0; w < NW; ++w) left -= s_ll[w];
  // rank of j under (frac descending, head index ascending)
  for (int j = tid; j < m; j += NT) {
    const double fj = frac[j];
    const int kj = who[j];
    int rank = 0;
    for (int i = 0; i < m; ++i) rank += (frac[i] > fj) || (frac[i] == fj && who[i] < kj);
    order[rank] = j;
    if (left >= 0) add[kj] += left / m + (rank < (int)(left % m) ? 1 : 0);
  }
  __syncthreads();
  if (left < 0 && tid == 0) {  // over-given by rounding: take back from the smallest fractions
    for (long long j = m - 1; left < 0; --j) {
      if (j < 0) j = m - 1;
      const int k = who[order[j]];
      if (add[k] > 0) { add[k] -= 1; ++left; }
    }
  }
  __syncthreads();
}

// Algorithm 2, one CTA per sequence:
//   eta_i = sum_j A_ij / sum_j B_ij,  B'_i = B_total eta_i / sum_i eta_i,
//   eta_ij = A_ij / B_ij,             B'_ij = B'_i eta_ij / sum_j eta_ij,
// integerised: min_b per head is set aside, the rule divides the remainder by largest
// remainders so the budgets sum to B_total, heads above max_b are clamped and their excess
// shared among the rest in the same proportions.  sum_i eta_i = 0 keeps the budgets.
__global__ void __launch_bounds__(NT) alg2_kernel(const long long* Asum, int* budget, int L, int H,
                                                  long long B_total, int min_b, int max_b) {
  extern __shared__ __align__(16) unsigned char sm[];
  const int N = L * H, tid = threadIdx.x;
  double* a = reinterpret_cast<double*>(sm);
  double* x = a + N;
  double* frac = x + N;
  double* eta_l = frac + N;
  double* S_l = eta_l + L;
  long long* add = reinterpret_cast<long long*>(S_l + L);
  int* who = reinterpret_cast<int*>(add + N);
  int* order = who + N;
  __shared__ double s_d[2];
  __shared__ long long s_ll[NW + 1];
  __shared__ int s_red[NW + 1];
  const size_t base = (size_t)blockIdx.x * N;
  for (int k = tid; k < N; k += NT) {
    a[k] = __ddiv_rn((double)Asum[base + k], 4294967296.0);
    add[k] = 0;
    who[k] = k;
  }
  __syncthreads();
  for (int i = tid; i < L; i += NT) {
    double sa = 0.0, sb = 0.0, sl = 0.0;
    for (int j = 0; j < H; ++j) {
      const double bij = (double)budget[base + i * H + j];
      sa = __dadd_rn(sa, a[i * H + j]);
      sb = __dadd_rn(sb, bij);
      sl = __dadd_rn(sl, __ddiv_rn(a[i * H + j], bij));
    }
    eta_l[i] = __ddiv_rn(sa, sb);
    S_l[i] = sl;
  }
  __syncthreads();
  if (tid == 0) {
    double S = 0.0;
    for (int i = 0; i < L; ++i) S = __dadd_rn(S, eta_l[i]);
    s_d[1] = S;
  }
  __syncthreads();
  const double S = s_d[1];
  if (!(S > 0.0)) return;
  const long long R = B_total - (long long)N * min_b;
  for (int k = tid; k < N; k += NT) {
    const int i = k / H;
    const double layer_share = __ddiv_rn(__dmul_rn((double)R, eta_l[i]), S);
    const double head_part = (S_l[i] > 0.0)
        ? __ddiv_rn(__ddiv_rn(a[k], (double)budget[base + k]), S_l[i])
        : __ddiv_rn(1.0, (double)H);
    x[k] = __dmul_rn(layer_share, head_part);
  }
  __syncthreads();
  share_out(R, who, N, x, add, frac, order, s_d, s_ll);
  for (;;) {
    long long excess = 0;
    for (int k = tid; k < N; k += NT) {
      const long long b = (long long)min_b + add[k];
      if (b > max_b) { excess += b - max_b; add[k] = (long long)max_b - min_b; }
    }
    excess = (long long)warp_sum_u64((unsigned long long)excess);
    __syncthreads();
    if ((tid & 31) == 0) s_ll[tid >> 5] = excess;
    __syncthreads();
    excess = 0;
    for (int w = 0; w < NW; ++w) excess += s_ll[w];
    __syncthreads();
    if (excess == 0) break;
    int m = 0;
    for (int b0 = 0; b0 < N; b0 += NT) {   // ordered compaction of the heads still under the cap
      const int k = b0 + tid;
      const int flag = (k < N) && ((long long)min_b + add[k] < max_b);
      int tot;
      const int r = block_excl_scan(flag, s_red, tot);
      if (flag) who[m + r] = k;
      m += tot;
    }
    __syncthreads();
    if (m == 0) break;
    share_out(excess, who, m, x, add, frac, order, s_d, s_ll);
  }
  for (int k = tid; k < N; k += NT) budget[base + k] = (int)(min_b + add[k]);
}

// ---------------------------------------------------------------------------------------
// Makes a head's list dense: the last entry moves into the hole an evicted entry left (one row and
// its metadata).  Needed before anything that works on a dense list outside a decode step.
__device__ __forceinline__ void close_hole(const State& st, int uid, int seq) {
  const int n = st.n_cur[uid], hole = st.hole[uid];
  __syncthreads();
  if (hole < n) {
    if (threadIdx.x < 32) move_entry(st, uid, seq, (size_t)uid * st.cap, hole, n, threadIdx.x);
    __syncthreads();
    if (threadIdx.x == 0) st.hole[uid] = n;
  }
  __syncthreads();
}

// Shrink pass for the heads of one layer (one CTA per head): a head holding more entries than
// its budget drops its lowest (decayed CRF, tau, pos) entries; the pages that become empty go
// back to the sequence's free list, from which heads that grew refill step by step.
__global__ void __launch_bounds__(NT) shrink_kernel(State st, int layer, int t_last, int* tmp, int tmp_stride) {
  __shared__ int sh[300];
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + layer) * st.H + head;
  const int n = st.n_cur[uid], B = st.budget[uid];
  if (n <= B || n < 2) return;
  close_hole(st, uid, seq);
  evict_many(st, uid, seq, n, min(n - B, n - 1), t_last, true, sh, tmp + (size_t)u * tmp_stride);
}

// ---------------------------------------------------------------------------------------
// Consistency check of page ownership: every pool page of a sequence must be owned exactly
// once, either by the free list or by one head, and every head must own the pages that back its
// entries and its hole.
__global__ void mark_free_kernel(State st, int* seen) {
  const int seq = blockIdx.y;
  const int top = st.free_top[seq];
  const int* stack = st.free_stack + (size_t)seq * st.pages_per_seq;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < top; i += (long long)gridDim.x * blockDim.x) {
    const int s = stack[i];
    if (s < 0 || s >= st.pages_per_seq) atomicAdd(&seen[(size_t)st.batch * st.pages_per_seq], 1);
    else atomicAdd(&seen[(size_t)seq * st.pages_per_seq + s], 1);
  }
}

__global__ void mark_owned_kernel(State st, int layer, int* seen) {
  const int u = blockIdx.x, seq = u / st.H, head = u % st.H;
  const int uid = (seq * st.L + layer) * st.H + head;
  const int own = st.npages[uid];
  if (threadIdx.x == 0) {
    const int n = st.n_cur[uid], hole = st.hole[uid];
    if (own * GRP <= n || own > st.capg || hole < 0 || hole > n) atomicAdd(&seen[(size_t)st.batch * st.pages_per_seq], 1);
  }
  for (int j = threadIdx.x; j < min(own, st.capg); j += blockDim.x) {
    const int s = st.ptab[(size_t)uid * st.capg + j];
    if (s < 0 || s >= st.pages_per_seq) atomicAdd(&seen[(size_t)st.batch * st.pages_per_seq], 1);
    else atomicAdd(&seen[(size_t)seq * st.pages_per_seq + s], 1);
  }
}

__global__ void count_bad_kernel(const int* seen, long long total, int* bad) {
  int loc = 0;
  for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
    loc += (seen[i] != 1);
  loc = warp_sum_i(loc);
  if ((threadIdx.x & 31) == 0 && loc) atomicAdd(bad, loc);
}

// ---------------------------------------------------------------------------------------
// State of one head for the host, entry by entry in list order (the hole skipped): records
// {position, CRF bits, tau} and, when asked for, the K and V rows in plain row layout.
__global__ void __launch_bounds__(NT) export_unit_kernel(State st, int uid, int seq, int* rec, unsigned char* krows,
                                                         unsigned char* vrows, int* n_out) {
  const int n = st.n_cur[uid], hole = st.hole[uid];
  const size_t mb = (size_t)uid * st.cap;
  if (threadIdx.x == 0) *n_out = n;
  for (int x = threadIdx.x; x < n; x += NT) {
    const int i = live_pos(x, hole);
    rec[3 * x] = st.meta_pos[mb + i];
    rec[3 * x + 1] = __float_as_int(st.meta_crf[mb + i]);
    rec[3 * x + 2] = st.meta_tau[mb + i];
  }
  if (!krows) return;
  const int c = threadIdx.x & 31;
  for (int x = threadIdx.x >> 5; x < n; x += NW) {
    const uint4 v = *reinterpret_cast<const uint4*>(entry_chunk(st, uid, seq, live_pos(x, hole), c));
    *reinterpret_cast<uint4*>((c < 16 ? krows : vrows) + (size_t)x * ROW_BYTES + (c & 15) * 16) = v;
  }
}

// The inverse: replaces the head's content by n entries given as records and rows (in any
// order; they become list positions 0 .. n-1), returns the pages it no longer needs and takes
// those it lacks.  One CTA; no other kernel that takes or returns pages runs beside it.
__global__ void __launch_bounds__(NT) import_unit_kernel(State st, int uid, int seq, const int* rec, const unsigned char* krows,
                                                         const unsigned char* vrows, int n, int budget) {
  __shared__ int s_base;
  const int tid = threadIdx.x;
  const int need = n / GRP + 1;
  int have = st.npages[uid];
  if (n + 1 > st.cap) {
    if (tid == 0) atomicOr(st.errword, ERR_CAPACITY);
    return;
  }
  if (have > need) {
    release_pages(st, uid, seq, n, &s_base);
  } else if (have < need) {
    if (tid == 0) {
      int top = atomicSub(&st.free_top[seq], need - have);
      if (top < need - have) {
        atomicAdd(&st.free_top[seq], need - have);
        atomicOr(st.errword, ERR_FREE_UNDERFLOW);
        top = -1;
      }
      s_base = top;
    }
    __syncthreads();
    if (s_base < 0) return;
    const int* stack = st.free_stack + (size_t)seq * st.pages_per_seq;
    for (int j = tid; j < need - have; j += NT) st.ptab[(size_t)uid * st.capg + have + j] = stack[s_base - 1 - j];
    __syncthreads();
    if (tid == 0) st.npages[uid] = need;
  }
  __syncthreads();
  const size_t mb = (size_t)uid * st.cap;
  for (int i = tid; i < n; i += NT) {
    st.meta_pos[mb + i] = rec[3 * i];
    st.meta_crf[mb + i] = __int_as_float(rec[3 * i + 1]);
    st.meta_tau[mb + i] = rec[3 * i + 2];
  }
  const int c = tid & 31;
  for (int i = tid >> 5; i < n; i += NW) {
    const uint4 v = *reinterpret_cast<const uint4*>((c < 16 ? krows : vrows) + (size_t)i * ROW_BYTES + (c & 15) * 16);
    *reinterpret_cast<uint4*>(entry_chunk(st, uid, seq, i, c)) = v;
  }
  if (tid == 0) { st.n_cur[uid] = n; st.hole[uid] = n; st.budget[uid] = budget; }
}

}  // namespace ckv
