// Decode attention of one layer (Section 2.2): the G queries of every kv head over its paged
// cache, split-K over the warps of a persistent grid.
//
// The layer's launch plan (plan.cuh) gives every warp its pieces: a piece is a range of the 16-key
// groups of one head (usually one piece per warp; several whole heads when there are more heads
// than warps).  A group is one pool page: 16 entries (K row + V row each) in 8 KB, stored so that
// the page, copied as it is into a ring stage by ONE bulk asynchronous copy, is read by ldmatrix
// without bank conflicts.  A warp keeps its ring of STAGES pages full across piece boundaries
// (the copies only need the cache, not the queries), waits for a stage on its mbarrier, and runs
// both contractions on the tensor cores with keys on the MMA M dimension and the (padded) query
// heads on N = 8:   S[16 keys x 8 heads] = K Q^T,   O^T[128 x 8 heads] += V^T P^T.
// A head that is one piece is written out directly.  A head whose pieces sit in consecutive warps
// of this CTA (the plan arranges that and marks it) is merged in shared memory: every warp leaves
// its (m, l, O) partial in its idle ring stages, the head's warps meet at a named barrier and
// share the query heads.  A head of more than eight pieces is merged that way run by run (whole
// CTAs and one shorter run) and its runs' partials through global memory: the warp whose ticket
// completes the head merges them into `out`; so is a head that the plan could not keep together
// (after the warp's own pieces, if it has more).  The arriving token is written into the head's hole (the place
// an evicted entry left, or the end of the list) by the warp that streams that group.  The scaled
// logits of the step are left in the scratch for the LRFU kernel, which marks hits from the final
// softmax weights without reading the cache again; the lines of the metadata that kernel will
// read are asked into L2 on the way.
#pragma once
#include "common.cuh"

namespace ckv {

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movm_t(uint32_t x) {
  uint32_t y;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while the kernel before it in the stream still runs; pdl_wait() returns once that
// kernel has completed and its writes are visible, pdl_launch() lets the kernel after this
// one start.  Both are no-ops for a launch without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;\n" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}\n"
               : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
// Bulk copy global -> shared with an L2 eviction policy for the lines it touches: 16-byte aligned
// addresses, size a multiple of 16; completion is counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
// Cache pages are read once per step and the whole cache is far larger than L2: they should
// leave L2 first.  The step's logits are read back by the LRFU kernel a little later: last.
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;\n" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void st_f32x2_hint(float* p, float a, float b, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v2.f32 [%0], {%1, %2}, %3;\n" ::"l"(p), "f"(a), "f"(b), "l"(pol) : "memory");
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;\n" : "=l"(t));
  return t;
}
// Waits for a stage's copy, for about a second at most: a copy that never lands raises the
// error word instead of hanging the GPU.  Returns false on that time-out.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > 1000000000ull) return false;
  }
}

// Named barriers 1..NW: the warps that hold the pieces of one head meet there.
__device__ __forceinline__ void bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;\n" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void bar_arrive(int id, int nthreads) {
  asm volatile("bar.arrive %0, %1;\n" ::"r"(id), "r"(nthreads) : "memory");
}

constexpr float LAZY = 8.0f;   // the running maximum (log2 domain) may trail the true one by this much

// The merge of HB heads over at most PB pieces in one round of loads: every lane loads the
// pieces' (m, l) itself (broadcast loads) next to its 4 channels of every O row, so nothing
// waits for a header round.  mm, L: merged reference point and normaliser per head.
template <int HB, int PB>
__device__ __forceinline__ void merge_small(const float* pbase, int PS, int npieces, int g0, int G, int lane,
                                            float (&mm)[HB], float (&L)[HB], float4 (&acc)[HB]) {
  float4 v[HB][PB];
  float pm[HB][PB], pl[HB][PB];
#pragma unroll
  for (int j = 0; j < PB; ++j) {
    const bool okp = j < npieces;
    const float* pp = pbase + (size_t)j * PS;
#pragma unroll
    for (int h = 0; h < HB; ++h) {
      const bool ok = okp && g0 + h < G;
      pm[h][j] = ok ? __ldcg(pp + g0 + h) : -INFINITY;
      pl[h][j] = ok ? __ldcg(pp + 8 + g0 + h) : 0.f;
      v[h][j] = ok ? __ldcg(reinterpret_cast<const float4*>(pp + 16 + (g0 + h) * HD) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
#pragma unroll
  for (int h = 0; h < HB; ++h) {
    float m = pm[h][0];
#pragma unroll
    for (int j = 1; j < PB; ++j) m = fmaxf(m, pm[h][j]);
    mm[h] = m;
    float l = 0.f;
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int j = 0; j < PB; ++j) {
      const float c = (pm[h][j] > -INFINITY) ? ex2(pm[h][j] - m) : 0.f;
      l = fmaf(pl[h][j], c, l);
      a.x = fmaf(v[h][j].x, c, a.x); a.y = fmaf(v[h][j].y, c, a.y);
      a.z = fmaf(v[h][j].z, c, a.z); a.w = fmaf(v[h][j].w, c, a.w);
    }
    L[h] = l;
    acc[h] = a;
  }
}

// out = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m) over the npieces partials of head u, by one warp.
__device__ __forceinline__ void merge_head(const DecodeParams& p, int u, int npieces, int lane) {
  const int G = p.G, PS = 16 + G * HD;
  const float* pbase = p.sc.partials + (size_t)u * p.sc.pmax * PS;
  auto put = [&](int g, float m, float L, const float4& a) {   // one head's result
    if (g < G) {
      const float iv = 1.0f / L;
      uint2 pk;
      pk.x = pack_bf16(a.x * iv, a.y * iv);
      pk.y = pack_bf16(a.z * iv, a.w * iv);
      *reinterpret_cast<uint2*>(p.out + ((size_t)(u * G + g)) * HD + lane * 4) = pk;
      if (lane == 0 && p.track) {   // reference point and normaliser of the step's softmax, for the LRFU kernel
        p.sc.mfin[u * (2 * QH) + g] = m;
        p.sc.mfin[u * (2 * QH) + QH + g] = L;
      }
    }
  };
  if (npieces <= 4) {   // the usual case: one round of loads for up to five heads
    if (G <= 5) {
      float mm[5], L[5];
      float4 acc[5];
      merge_small<5, 4>(pbase, PS, npieces, 0, G, lane, mm, L, acc);
#pragma unroll
      for (int h = 0; h < 5; ++h) put(h, mm[h], L[h], acc[h]);
    } else {
      for (int g0 = 0; g0 < G; g0 += 4) {
        float mm[4], L[4];
        float4 acc[4];
        merge_small<4, 4>(pbase, PS, npieces, g0, G, lane, mm, L, acc);
#pragma unroll
        for (int h = 0; h < 4; ++h) put(g0 + h, mm[h], L[h], acc[h]);
      }
    }
  } else {   // four heads x four pieces per round of loads, rounds chained by the usual rescale
    for (int g0 = 0; g0 < G; g0 += 4) {
      float mg[4], Lg[4];
      float4 acc[4];
#pragma unroll
      for (int h = 0; h < 4; ++h) { mg[h] = -INFINITY; Lg[h] = 0.f; acc[h] = make_float4(0.f, 0.f, 0.f, 0.f); }
      for (int pc0 = 0; pc0 < npieces; pc0 += 4) {
        float mm[4], L[4];
        float4 a2[4];
        merge_small<4, 4>(pbase + (size_t)pc0 * PS, PS, npieces - pc0, g0, G, lane, mm, L, a2);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
          const float mn = fmaxf(mg[h], mm[h]);
          const float ca = (mg[h] > -INFINITY) ? ex2(mg[h] - mn) : 0.f, cb = (mm[h] > -INFINITY) ? ex2(mm[h] - mn) : 0.f;
          Lg[h] = Lg[h] * ca + L[h] * cb;
          acc[h].x = acc[h].x * ca + a2[h].x * cb; acc[h].y = acc[h].y * ca + a2[h].y * cb;
          acc[h].z = acc[h].z * ca + a2[h].z * cb; acc[h].w = acc[h].w * ca + a2[h].w * cb;
          mg[h] = mn;
        }
      }
#pragma unroll
      for (int h = 0; h < 4; ++h) put(g0 + h, mg[h], Lg[h], acc[h]);
    }
  }
}

__global__ void __maxnreg__(160) attn_kernel(const DecodeParams p) {   // (160 registers: two LRFU CTAs fit beside it on an SM)
  extern __shared__ __align__(1024) unsigned char smem[];
  const State& st = p.st;
  // Without `early` the kernel before this one may still be writing the lists this one reads.
  if (!p.early) pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  // ring stages, then one mbarrier per stage, then every warp's queue of fetched pieces
  const uint32_t bars_u32 = smem_u32(smem) + RING_BYTES;
  int* fifo = reinterpret_cast<int*>(smem + RING_BYTES + NW * STAGES * 8) + w * FIFO;
  if (tid < NW * STAGES) mbar_init(bars_u32 + tid * 8, 1);
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");   // made visible to the copy engine
  __syncthreads();
  const int4 range = __ldg(p.plan.wrange + blockIdx.x * NW + w);   // (requested together with the header)
  if (__ldg(p.plan.hdr + 2) != (int)gridDim.x * NW || __ldg(p.plan.hdr + 3) != p.append) {   // a plan made for another launch
    if (tid == 0 && blockIdx.x == 0) atomicOr(st.errword, ERR_PLAN);
    return;
  }
  if (range.x >= range.y) return;   // no run for this warp

  const int G = p.G, PS = 16 + G * HD;
  const uint32_t ring_u32 = smem_u32(smem) + w * (STAGES * PAGE_BYTES);
  const uint32_t bar0 = bars_u32 + w * (STAGES * 8);
  const int gid = lane >> 2, tig = lane & 3, mi = lane >> 3, r8 = lane & 7;
  const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
  // ldmatrix row addresses inside a stage: entry row r, 16-byte chunk c at 512 r + 16 (c ^ (r & 7))
  const uint32_t krow = (uint32_t)(((mi & 1) * 8 + r8) * SLOT_BYTES), khalf = (uint32_t)(mi >> 1);
  const uint32_t vrow = (uint32_t)(((mi >> 1) * 8 + r8) * SLOT_BYTES), vhalf = (uint32_t)(mi & 1);
  bool waited = p.early == 0;
  uint32_t phases = 0;      // bit s: parity of the next completion of stage s
  int fsi = 0, csi = 0;     // stage the next copy fills / the next compute reads
  int fq_head = 0, fq_tail = 0;
  int defer0 = -1, defer1 = -1;   // heads this warp completed and merges after its own run

  // ---- fetching side: the piece whose groups are being requested
  int f_pi = range.x, f_next = 0, f_hi = 0, f_ntot = 0, f_seq = 0, ids = 0, idbase = 0;
  const int* pt = st.ptab;
  auto entries_of = [&](int u) {   // entries of head u that take part in this launch
    const int uid = ((u / st.H) * st.L + p.layer) * st.H + (u % st.H);
    int n = __ldg(st.n_cur + uid);
    if (p.n_limit > 0) n = min(n, p.n_limit);
    return n + p.append;
  };
  // the descriptor of the warp's first piece came with its range
  const int4 dd_first = range.z >= 0 ? make_int4(range.z, range.w & 4095, (range.w >> 12) & 4095, range.w >> 24)
                                     : __ldg(p.plan.desc + range.x);
  auto open_piece = [&](int pi, const int4 dd) {
    const int u = dd.x;
    f_seq = u / st.H;
    f_ntot = entries_of(u);
    {   // piece dd.y of dd.z over the head's groups as they are now
      const unsigned g = (unsigned)(f_ntot + GRP - 1) / GRP;
      f_next = (int)(g * (unsigned)dd.y / (unsigned)dd.z);
      f_hi = (int)(g * (unsigned)(dd.y + 1) / (unsigned)dd.z);
    }
    const int f_uid = (f_seq * st.L + p.layer) * st.H + (u % st.H);
    pt = st.ptab + (size_t)f_uid * st.capg;
    if (p.track) {
      // The LRFU kernel that follows reads position, tau and CRF of these entries while the next
      // layer's attention saturates HBM, and every round trip to DRAM costs it microseconds then:
      // their lines are asked into L2 now (12 bytes per entry against the 512 streamed here).
      const size_t e0 = (size_t)f_uid * st.cap + (size_t)f_next * GRP, e1 = (size_t)f_uid * st.cap + (size_t)f_hi * GRP;
      const char* bases[3] = {reinterpret_cast<const char*>(st.meta_pos), reinterpret_cast<const char*>(st.meta_tau),
                              reinterpret_cast<const char*>(st.meta_crf)};
      const int nl = (int)(((e1 * 4 + 127) >> 7) - ((e0 * 4) >> 7));   // 128-byte lines per array (arrays are 256-byte aligned)
      for (int x = lane; x < 3 * nl; x += 32) {
        const char* a = bases[x / nl] + (((e0 * 4) >> 7) + (x % nl)) * 128;
        asm volatile("prefetch.global.L2::evict_last [%0];\n" ::"l"(a));
      }
    }
    idbase = f_next;
    ids = (f_next + lane < f_hi) ? __ldg(pt + f_next + lane) : 0;   // page ids of groups f_next + lane
    if (lane == 0) fifo[fq_tail & (FIFO - 1)] = pi;
    ++fq_tail;
    __syncwarp();
  };
  auto fetch_next = [&]() -> bool {
    if (f_pi < 0) return false;
    if (f_next == f_hi) {
      f_pi = (f_pi + 1 < range.y) ? f_pi + 1 : -1;
      if (f_pi < 0) return false;
      open_piece(f_pi, __ldg(p.plan.desc + f_pi));
    }
    if (f_next - idbase >= 32) { idbase = f_next; ids = (f_next + lane < f_hi) ? __ldg(pt + f_next + lane) : 0; }
    const int page = __shfl_sync(0xffffffffu, ids, f_next - idbase);
    const int valid = min(GRP, f_ntot - f_next * GRP);
    const uint32_t stage = ring_u32 + fsi * PAGE_BYTES;
    if (valid < GRP) {   // rows past the head's end must not feed stale bits into the MMAs
      for (int e = valid; e < GRP; ++e)
        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(stage + e * SLOT_BYTES + lane * 16), "r"(0) : "memory");
      asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      __syncwarp();
    }
    if (lane == 0) {
      const uint32_t bar = bar0 + fsi * 8;
      mbar_expect_tx(bar, (uint32_t)valid * SLOT_BYTES);
      bulk_g2s_hint(stage, st.pool + ((size_t)f_seq * st.pages_per_seq + (unsigned)page) * PAGE_BYTES,
                    (uint32_t)valid * SLOT_BYTES, bar, pol_stream);
    }
    ++f_next;
    fsi = (fsi + 1 == STAGES) ? 0 : fsi + 1;
    return true;
  };
  open_piece(f_pi, dd_first);
#pragma unroll 1
  for (int s = 0; s < STAGES; ++s) fetch_next();
  // everything above reads only the cache, its lists and the plan; the call's inputs (q, the
  // arriving rows) may come from the kernel ahead in the stream
  if (!waited) { pdl_wait(); waited = true; }
  pdl_launch();

  // ---- computing side: one piece after the other, in the order they were fetched
#pragma unroll 1
  while (fq_head != fq_tail) {
    const int pi = fifo[fq_head & (FIFO - 1)];
    ++fq_head;
    const int4 dd = pi == range.x ? dd_first : __ldg(p.plan.desc + pi);
    const int u = dd.x, piece = dd.y, npieces = dd.z;
    const int seq = u / st.H;
    const int uid = (seq * st.L + p.layer) * st.H + (u % st.H);
    const int n_tot = entries_of(u);
    const unsigned g_u = (unsigned)(n_tot + GRP - 1) / GRP;
    const int lo = (int)(g_u * (unsigned)piece / (unsigned)npieces), hi = (int)(g_u * (unsigned)(piece + 1) / (unsigned)npieces);
    const int hole = p.append ? __ldg(st.hole + uid) : -1;   // where the arriving token goes
    // A head whose pieces all belong to consecutive warps of this CTA, each warp holding nothing else
    // (the plan marks it), is merged through shared memory.
    // (A head of more than eight pieces is placed in runs of eight, whole CTAs and one shorter run:
    // every run is merged in its CTA, and only one partial per run goes through global memory.)
    const bool runs = dd.w == 2;
    const int jr = runs ? (piece & (NW - 1)) : piece;                       // this piece's place in its run
    const int rl = runs ? min(NW, npieces - (piece & ~(NW - 1))) : npieces;   // pieces in the run
    const int first_w = w - jr;
    const bool local = dd.w != 0 && npieces > 1 && range.y - range.x == 1 && first_w >= 0 && first_w + rl <= NW;
    // the G queries as B fragments, running softmax state, O^T accumulators
    uint32_t qb[8][2];
    {
      const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q + ((size_t)u * G + gid) * HD);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        qb[ks][0] = (gid < G) ? q32[ks * 8 + tig] : 0u;
        qb[ks][1] = (gid < G) ? q32[ks * 8 + tig + 4] : 0u;
      }
    }
    float o[8][4];
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float* lrow0 = p.sc.logits + (size_t)u * p.sc.cap_s * QH + gid * QH + 2 * tig;

#pragma unroll 1
    for (int ci = lo; ci < hi; ++ci) {
      if (!mbar_wait_bounded(bar0 + csi * 8, (phases >> csi) & 1u)) {
        // a copy did not land: flag it, give the other stages' copies their chance to land in
        // this CTA's memory while it still belongs to us, and leave the run unfinished
        if (lane == 0) atomicOr(st.errword, ERR_COPY_TIMEOUT);
        for (int s = 0; s < STAGES; ++s)
          if (s != csi) mbar_wait_bounded(bar0 + s * 8, (phases >> s) & 1u);
        if (local) bar_arrive(1 + first_w, 32 * rl);   // the run's other warps must not wait for this one
        return;
      }
      phases ^= 1u << csi;
      const uint32_t stage = ring_u32 + csi * PAGE_BYTES;
      const int base = ci * GRP;
      const int valid = min(GRP, n_tot - base);
      if (hole >= base && hole < base + GRP) {
        // the arriving token: chunk `lane` of its K row (lanes 0..15) or V row (16..31) goes into the
        // stage and into the head's page, at the place the hole has in both
        const unsigned char* src = reinterpret_cast<const unsigned char*>(lane < 16 ? p.k_new : p.v_new) +
                                   (size_t)u * ROW_BYTES + (lane & 15) * 16;
        const uint4 val = *reinterpret_cast<const uint4*>(src);
        const int off = chunk_offset(hole - base, lane);
        asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};\n" ::"r"(stage + off), "r"(val.x), "r"(val.y), "r"(val.z), "r"(val.w) : "memory");
        const int page = __ldg(st.ptab + (size_t)uid * st.capg + ci);
        *reinterpret_cast<uint4*>(st.pool + ((size_t)seq * st.pages_per_seq + page) * PAGE_BYTES + off) = val;
        if (lane == 0) {
          const size_t mb = (size_t)uid * st.cap;
          st.meta_pos[mb + hole] = p.t;
          st.meta_tau[mb + hole] = p.t;
          st.meta_crf[mb + hole] = 0.0f;
        }
      }
      __syncwarp();   // zero rows and the arriving row other lanes stored are visible
      // ---- S[key][head] = K Q^T over the 8 k-steps of 16 channels, two chains of four
      float s[4] = {0.f, 0.f, 0.f, 0.f};
      {
        float s2[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t ka = stage + krow;
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
          uint32_t a[4], a2[4];
          ldsm_x4(a, ka + (((2 * ks + khalf) ^ r8) << 4));
          ldsm_x4(a2, ka + (((2 * ks + 2 + khalf) ^ r8) << 4));
          mma_bf16(s, a, qb[ks][0], qb[ks][1]);
          mma_bf16(s2, a2, qb[ks + 1][0], qb[ks + 1][1]);
        }
#pragma unroll
        for (int x = 0; x < 4; ++x) s[x] += s2[x];
      }
      const bool v0 = gid < valid, v1 = gid + 8 < valid;
      if (p.track) {
        float* lrow = lrow0 + (size_t)base * QH;
        if (v0) st_f32x2_hint(lrow, __fmul_rn(s[0], p.scale), __fmul_rn(s[1], p.scale), pol_keep);
        if (v1) st_f32x2_hint(lrow + 8 * QH, __fmul_rn(s[2], p.scale), __fmul_rn(s[3], p.scale), pol_keep);
      }
      // ---- online softmax, this lane's two heads (2 tig, 2 tig + 1) over its two keys
      const float t0 = v0 ? s[0] * p.scale_log2 : -INFINITY, t1 = v0 ? s[1] * p.scale_log2 : -INFINITY;
      const float t2 = v1 ? s[2] * p.scale_log2 : -INFINITY, t3 = v1 ? s[3] * p.scale_log2 : -INFINITY;
      float c0 = fmaxf(t0, t2), c1 = fmaxf(t1, t3);
#pragma unroll
      for (int x = 4; x < 32; x <<= 1) {
        c0 = fmaxf(c0, __shfl_xor_sync(0xffffffffu, c0, x));
        c1 = fmaxf(c1, __shfl_xor_sync(0xffffffffu, c1, x));
      }
      // the reference point only moves when a maximum has grown by more than LAZY, so most groups
      // skip the rescale; weights stay below 2^LAZY
      if (__any_sync(0xffffffffu, c0 > m0 + LAZY || c1 > m1 + LAZY)) {
        const float n0 = fmaxf(m0, c0), n1 = fmaxf(m1, c1);
        const float r0 = ex2(m0 - n0), r1 = ex2(m1 - n1);
        l0 *= r0; l1 *= r1;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= r0; o[mt][1] *= r1; o[mt][2] *= r0; o[mt][3] *= r1; }
        m0 = n0; m1 = n1;
      }
      const float p0 = ex2(t0 - m0), p1 = ex2(t1 - m1), p2 = ex2(t2 - m0), p3 = ex2(t3 - m1);
      l0 += p0 + p2;
      l1 += p1 + p3;
      // P^T as the B operand: transpose the two 8 x 8 (key x head) blocks across the warp.  The
      // weights go in as a bf16 head plus a bf16 remainder, which keeps 16 bits of each.
      const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1), h23 = __floats2bfloat162_rn(p2, p3);
      const uint32_t b0 = movm_t(*reinterpret_cast<const uint32_t*>(&h01)), b1 = movm_t(*reinterpret_cast<const uint32_t*>(&h23));
      const uint32_t rr0 = movm_t(pack_bf16(p0 - __low2float(h01), p1 - __high2float(h01)));
      const uint32_t rr1 = movm_t(pack_bf16(p2 - __low2float(h23), p3 - __high2float(h23)));
      // ---- O^T[channel][head] += V^T P^T, 8 tiles of 16 channels
      {
        const uint32_t va = stage + vrow;
#pragma unroll
        for (int mt = 0; mt < 8; mt += 2) {   // two tiles at a time: the two MMAs of a tile depend on each other
          uint32_t a[4], a2[4];
          ldsm_x4_t(a, va + (((16 + 2 * mt + vhalf) ^ r8) << 4));
          ldsm_x4_t(a2, va + (((16 + 2 * mt + 2 + vhalf) ^ r8) << 4));
          mma_bf16(o[mt], a, b0, b1);
          mma_bf16(o[mt + 1], a2, b0, b1);
          mma_bf16(o[mt], a, rr0, rr1);
          mma_bf16(o[mt + 1], a2, rr0, rr1);
        }
      }
      csi = (csi + 1 == STAGES) ? 0 : csi + 1;
      __syncwarp();   // the stage is free again
      fetch_next();   // and is refilled at once, with the next group of this run
    }

    // l over the keys of all lanes that hold the same heads
    float ls0 = l0, ls1 = l1;
#pragma unroll
    for (int x = 4; x < 32; x <<= 1) {
      ls0 += __shfl_xor_sync(0xffffffffu, ls0, x);
      ls1 += __shfl_xor_sync(0xffffffffu, ls1, x);
    }
    const int h0 = 2 * tig, h1 = 2 * tig + 1;
    if (npieces == 1) {
      // ---- the whole head was this warp's: normalise and write `out` from the accumulators
      const float i0 = 1.0f / ls0, i1 = 1.0f / ls1;
      __nv_bfloat16* ob = p.out + (size_t)u * G * HD + gid;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        if (h0 < G) {
          ob[h0 * HD + 16 * mt] = __float2bfloat16_rn(o[mt][0] * i0);
          ob[h0 * HD + 16 * mt + 8] = __float2bfloat16_rn(o[mt][2] * i0);
        }
        if (h1 < G) {
          ob[h1 * HD + 16 * mt] = __float2bfloat16_rn(o[mt][1] * i1);
          ob[h1 * HD + 16 * mt + 8] = __float2bfloat16_rn(o[mt][3] * i1);
        }
      }
      if (gid == 0 && p.track) {   // reference point and normaliser of the step's softmax, for the LRFU kernel
        if (h0 < G) { p.sc.mfin[u * (2 * QH) + h0] = m0; p.sc.mfin[u * (2 * QH) + QH + h0] = ls0; }
        if (h1 < G) { p.sc.mfin[u * (2 * QH) + h1] = m1; p.sc.mfin[u * (2 * QH) + QH + h1] = ls1; }
      }
      continue;
    }
    if (local) {
      // ---- the piece's partial goes into this warp's ring (idle by now: its only piece is done);
      // after a barrier of the head's warps each of them merges a share of the query heads
      constexpr int HS = HD + 4;   // row stride that spreads the four head pairs of a store over the banks
      constexpr int WSTRIDE = STAGES * PAGE_BYTES;
      float* mine = reinterpret_cast<float*>(smem + w * WSTRIDE);
      if (gid == 0) {
        *reinterpret_cast<float2*>(mine + 2 * tig) = make_float2(m0, m1);
        *reinterpret_cast<float2*>(mine + 8 + 2 * tig) = make_float2(ls0, ls1);
      }
      {
        float* po = mine + 16 + gid;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          if (h0 < G) { po[h0 * HS + 16 * mt] = o[mt][0]; po[h0 * HS + 16 * mt + 8] = o[mt][2]; }
          if (h1 < G) { po[h1 * HS + 16 * mt] = o[mt][1]; po[h1 * HS + 16 * mt + 8] = o[mt][3]; }
        }
      }
      bar_sync(1 + first_w, 32 * rl);
      const unsigned char* base = smem + first_w * WSTRIDE;
      float* rpart = p.sc.partials + ((size_t)u * p.sc.pmax + (piece >> 3)) * PS;   // the run's partial (runs only)
      for (int g = jr; g < G; g += rl) {
        float pm[NW], pl[NW];
        float4 v[NW];
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < NW; ++j) {
          const float* pp = reinterpret_cast<const float*>(base + (j < rl ? j : 0) * WSTRIDE);
          pm[j] = (j < rl) ? pp[g] : -INFINITY;
          pl[j] = (j < rl) ? pp[8 + g] : 0.f;
          v[j] = *reinterpret_cast<const float4*>(pp + 16 + g * HS + lane * 4);
          m = fmaxf(m, pm[j]);
        }
        float L = 0.f;
        float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int j = 0; j < NW; ++j) {
          const float c = (pm[j] > -INFINITY) ? ex2(pm[j] - m) : 0.f;
          L = fmaf(pl[j], c, L);
          a.x = fmaf(v[j].x, c, a.x); a.y = fmaf(v[j].y, c, a.y);
          a.z = fmaf(v[j].z, c, a.z); a.w = fmaf(v[j].w, c, a.w);
        }
        if (runs) {   // the run's share of the head, not normalised
          *reinterpret_cast<float4*>(rpart + 16 + g * HD + lane * 4) = a;
          if (lane == 0) { rpart[g] = m; rpart[8 + g] = L; }
          continue;
        }
        const float iv = 1.0f / L;
        uint2 pk;
        pk.x = pack_bf16(a.x * iv, a.y * iv);
        pk.y = pack_bf16(a.z * iv, a.w * iv);
        *reinterpret_cast<uint2*>(p.out + ((size_t)(u * G + g)) * HD + lane * 4) = pk;
        if (lane == 0 && p.track) {
          p.sc.mfin[u * (2 * QH) + g] = m;
          p.sc.mfin[u * (2 * QH) + QH + g] = L;
        }
      }
      if (!runs) continue;
      // every warp of the head counts itself once its share of its run's partial is written; the
      // one that completes the count merges the runs
      __syncwarp();
      int last = 0;
      if (lane == 0) {
        int old;
        asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(p.sc.ticket + u) : "memory");
        last = (old == npieces - 1);
        if (last) p.sc.ticket[u] = 0;
      }
      last = __shfl_sync(0xffffffffu, last, 0);
      if (last) merge_head(p, u, (npieces + NW - 1) / NW, lane);
      continue;
    }
    // ---- publish the piece's partial and take a ticket
    float* part = p.sc.partials + ((size_t)u * p.sc.pmax + piece) * PS;
    if (gid == 0) {
      *reinterpret_cast<float2*>(part + 2 * tig) = make_float2(m0, m1);
      *reinterpret_cast<float2*>(part + 8 + 2 * tig) = make_float2(ls0, ls1);
    }
    {
      float* po = part + 16 + gid;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        if (h0 < G) { po[h0 * HD + 16 * mt] = o[mt][0]; po[h0 * HD + 16 * mt + 8] = o[mt][2]; }
        if (h1 < G) { po[h1 * HD + 16 * mt] = o[mt][1]; po[h1 * HD + 16 * mt + 8] = o[mt][3]; }
      }
    }
    // Release / acquire on the ticket: the warp barrier makes every lane's stores happen before
    // lane 0's atomic, whose release makes them visible to the warp that acquires the last ticket.
    __syncwarp();
    int last = 0;
    if (lane == 0) {
      int old;
      asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;\n" : "=r"(old) : "l"(p.sc.ticket + u) : "memory");
      last = (old == npieces - 1);
      if (last) p.sc.ticket[u] = 0;   // ready for the next launch that uses this scratch set
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) continue;
    // the head is complete.  Merging it now would stall this warp's stream for a round trip to L2,
    // so a warp with more of its run ahead merges afterwards (a run cuts at most two heads).
    if (fq_head != fq_tail && defer0 < 0) defer0 = u;
    else if (fq_head != fq_tail && defer1 < 0) defer1 = u;
    else merge_head(p, u, npieces, lane);
  }
  if (defer0 >= 0) merge_head(p, defer0, __ldg(p.plan.npc + defer0), lane);
  if (defer1 >= 0) merge_head(p, defer1, __ldg(p.plan.npc + defer1), lane);
}

}  // namespace ckv
