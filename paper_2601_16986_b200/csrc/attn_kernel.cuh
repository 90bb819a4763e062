// Decode attention of one layer (Section 2.2): the G queries of every kv head over its
// slot-indexed cache, split-K over the warps of a persistent grid.
//
// Every kv head of the layer is cut into nearly equal pieces of 16-key groups, as many as its
// share of the grid's warps, and every warp streams one piece (more when there are more heads
// than warps) through a private ring of shared-memory stages.
// A stage holds 16 entries; every entry (K row + V row, the 512 contiguous bytes of its pool
// slot) arrives by one bulk asynchronous copy issued by the lane that holds its slot id and is
// counted by the stage's mbarrier, so there is no block-wide barrier after the prologue.  Both
// contractions run on the tensor cores with keys on the MMA M dimension and the (padded)
// query heads on N = 8:   S[16 keys x 8 heads] = K Q^T,   O^T[128 x 8 heads] += V^T P^T.
// A warp publishes the (m, l, O) partial of its piece; the warp whose partial completes a
// head merges them into `out`.  The scaled logits of the step are left in the
// scratch for the LRFU kernel, which marks hits from the final softmax weights without
// reading the cache again.
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

// A stage is 16 rows of ENTRY_STRIDE bytes: K row, V row, 16 bytes of padding.  The odd multiple
// of 16 bytes puts the eight rows an ldmatrix touches into eight different bank groups.
constexpr int ENTRY_STRIDE = SLOT_BYTES + 16;
static_assert(STAGE_BYTES == GRP * ENTRY_STRIDE, "stage size");

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
// Bulk copy global -> shared: 16-byte aligned addresses, size a multiple of 16; completion is
// counted in bytes on `bar`.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];\n"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// The same with an L2 eviction policy for the lines it touches.
__device__ __forceinline__ void bulk_g2s_hint(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;\n"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar), "l"(pol) : "memory");
}
// Cache rows are read once per step and the whole cache is far larger than L2: they should
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
// Waits for a stage's copies, for about a second at most: a copy that never lands raises the
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

constexpr int MAX_STAGES = 12;  // a warp's ring never grows beyond this
constexpr int PIECE_SOFT = 24;  // groups a piece may grow to when that saves merge rounds
constexpr float LAZY = 8.0f;   // the running maximum (log2 domain) may trail the true one by this much

// Accumulates HB heads x PB pieces of split-K partials for 4 output channels per lane; every
// load is issued before the first is consumed.
template <int HB, int PB>
__device__ __forceinline__ void merge_rows(const float* pbase, int PS, int npieces, int pc0, int g0, int G,
                                           int lane, const float (&mg)[HB], float4 (&acc)[HB]) {
  float4 v[HB][PB];
  float sc[HB][PB];
#pragma unroll
  for (int j = 0; j < PB; ++j) {
    const bool okp = pc0 + j < npieces;
    const float* pp = pbase + (size_t)(pc0 + j) * PS;
#pragma unroll
    for (int h = 0; h < HB; ++h) {
      const bool ok = okp && g0 + h < G;
      sc[h][j] = ok ? __ldcg(pp + g0 + h) : -INFINITY;
      v[h][j] = ok ? __ldcg(reinterpret_cast<const float4*>(pp + 16 + (g0 + h) * HD) + lane) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
#pragma unroll
  for (int j = 0; j < PB; ++j)
#pragma unroll
    for (int h = 0; h < HB; ++h) {
      const float c = ex2(sc[h][j] - mg[h]);
      acc[h].x = fmaf(v[h][j].x, c, acc[h].x); acc[h].y = fmaf(v[h][j].y, c, acc[h].y);
      acc[h].z = fmaf(v[h][j].z, c, acc[h].z); acc[h].w = fmaf(v[h][j].w, c, acc[h].w);
    }
}

// The whole merge of HB heads over at most PB pieces in one round of loads: every lane loads
// the pieces' (m, l) itself (broadcast loads) next to its 4 channels of every O row, so nothing
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

// The streaming of a warp's pieces.  DEEP: the CTA's ring stages are shared out among at most two
// warps, the last stage of a warp's share holds the slot ids of its piece (one bulk copy of the
// list segment), so that no copy waits for a global load of ids.  Otherwise: three stages per
// warp, ids requested through registers two fires ahead.
template <bool DEEP>
__device__ __forceinline__ void stream_pieces(const DecodeParams& p, unsigned char* smem, const int* off, const int* nin,
                                              int U, int Ptot, int nWarps, int nall_rt, bool dyn, int pi, uint32_t bars_u32,
                                              int chunk0) {
  const State& st = p.st;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int G = p.G;
  const int PS = 16 + G * HD;
  const int nall = DEEP ? nall_rt : STAGES;
  constexpr bool ids_in_smem = DEEP;
  const int nst = DEEP ? nall - 1 : STAGES;   // ring depth per working warp
  (void)tid;
  const uint32_t ring_u32 = smem_u32(smem) + w * (nall * STAGE_BYTES);   // w < apc whenever the warp has a piece
  const uint32_t ids_u32 = ring_u32 + nst * STAGE_BYTES;
  const uint32_t idbar = bars_u32 + (NW * STAGES + w) * 8;
  uint32_t idphase = 0;
  const int gid = lane >> 2, tig = lane & 3;
  const int mi = lane >> 3, r8 = lane & 7;
  const uint32_t bar0 = bars_u32 + w * (nall * 8);
  // ldmatrix row addresses inside a stage: K tile of k-step ks at kb + 32 ks, V tile of channel
  // tile mt at vb + 32 mt
  const uint32_t kb = (uint32_t)(((mi & 1) * 8 + r8) * ENTRY_STRIDE + (mi >> 1) * 16);
  const uint32_t vb = (uint32_t)(ROW_BYTES + ((mi >> 1) * 8 + r8) * ENTRY_STRIDE + (mi & 1) * 16);

  const uint64_t pol_stream = policy_evict_first(), pol_keep = policy_evict_last();
  int fsi = 0, csi = 0;     // stage the next fire fills / the next compute reads
  uint32_t phases = 0;      // bit s: parity of the next completion of stage s
  bool waited = p.early == 0;

#pragma unroll 1
  for (; pi < Ptot; pi += (dyn ? Ptot : nWarps)) {
    // ---- the piece: head u, groups [lo, hi) of its list
    int u;
    {
      int a = 0, b = U;
      while (b - a > 1) {
        const int mid = (a + b) >> 1;
        if (off[mid] <= pi) a = mid; else b = mid;
      }
      u = a;
    }
    const int seq = u / st.H, head = u % st.H;
    const int uid = (seq * st.L + p.layer) * st.H + head;
    const int n_old = nin[u], n_tot = n_old + p.append;
    const int g_u = (n_tot + GRP - 1) / GRP;
    const int piece = pi - off[u], npieces = off[u + 1] - off[u];
    // (32-bit products: g_u * npieces stays below 2^32 for any list that fits the pool)
    const int lo = (int)((unsigned)g_u * (unsigned)piece / (unsigned)npieces);
    const int hi = (int)((unsigned)g_u * (unsigned)(piece + 1) / (unsigned)npieces);
    // A head whose pieces all belong to this CTA is merged through shared memory.
    const int first_w = off[u] - chunk0;   // warp that streams the head's first piece
    const bool local = !DEEP && chunk0 >= 0 && npieces > 1 && first_w >= 0 && first_w + npieces <= NW;
    const size_t mb = (size_t)uid * st.cap;
    const int* list = st.list_slot + mb;
    const unsigned char* pool = st.pool + (size_t)seq * st.slots_per_seq * SLOT_BYTES;

    // ---- issuing side.  The lane that holds an entry's slot id issues its copy.  The ids come
    // from shared memory (deep rings) or are requested two fires before they are needed.
    auto slots_of = [&](int idx) {   // lane e: pool slot of entry 16 idx + e (0 past the end)
      const int i = idx * GRP + lane;
      return (lane < GRP && idx < hi && i < n_tot) ? list[i] : 0;
    };
    auto fire = [&](int idx, int slot, uint32_t stage, uint32_t bar) {
      const int valid = min(GRP, n_tot - idx * GRP);
      const int has_new = p.append && idx == g_u - 1;   // the head's last entry is the arriving token
      const int nv = valid - has_new;                   // entries that come from the pool
      if (lane == 0) mbar_expect_tx(bar, (uint32_t)valid * SLOT_BYTES);
      __syncwarp();
      if (lane < nv) bulk_g2s_hint(stage + lane * ENTRY_STRIDE, pool + (size_t)(unsigned)slot * SLOT_BYTES, SLOT_BYTES, bar, pol_stream);
      if (has_new) {   // it comes from the call's inputs
        if (!waited) { pdl_wait(); waited = true; }
        if (lane < 2)
          bulk_g2s(stage + nv * ENTRY_STRIDE + lane * ROW_BYTES,
                   reinterpret_cast<const unsigned char*>(lane == 0 ? p.k_new : p.v_new) + (size_t)u * ROW_BYTES,
                   ROW_BYTES, bar);
      }
      if (valid < GRP) {   // rows past the head's end must not feed garbage into the MMAs
        for (int e = valid; e < GRP; ++e)
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(stage + e * ENTRY_STRIDE + lane * 16), "r"(0) : "memory");
        asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory");
      }
    };
    // groups flow through the ring, nst-1 of them in flight
    int next = lo;
    int sl0 = 0, sl1 = 0;
    const bool ids_here = ids_in_smem && (hi - lo) * GRP * 4 <= STAGE_BYTES;   // else: ids through registers
    if (ids_here) {
      // the list positions of groups lo .. hi-1 are contiguous and 64-byte aligned
      if (lane == 0) {
        mbar_expect_tx(idbar, (uint32_t)(hi - lo) * GRP * 4);
        bulk_g2s(ids_u32, list + (size_t)lo * GRP, (uint32_t)(hi - lo) * GRP * 4, idbar);
      }
      if (!mbar_wait_bounded(idbar, idphase)) {
        if (lane == 0) atomicOr(st.errword, ERR_COPY_TIMEOUT);
        return;
      }
      idphase ^= 1u;
    } else {
      sl0 = slots_of(lo); sl1 = slots_of(lo + 1);
    }
    auto fire_next = [&]() {
      if (next < hi) {
        int slot = sl0;
        if (ids_here) {
          asm volatile("ld.shared.b32 %0, [%1];\n" : "=r"(slot) : "r"(ids_u32 + (uint32_t)((next - lo) * GRP + (lane & 15)) * 4));
        } else {
          sl0 = sl1;
          sl1 = slots_of(next + 2);
        }
        fire(next, slot, ring_u32 + fsi * STAGE_BYTES, bar0 + fsi * 8);
        ++next;
        fsi = (fsi + 1 == nst) ? 0 : fsi + 1;
      }
    };
#pragma unroll 1
    for (int s = 0; s < nst - 1; ++s) fire_next();
    // everything above reads only the cache and its lists; the call's inputs (q here, the
    // arriving row inside fire) may come from the kernel ahead in the stream
    if (!waited) { pdl_wait(); waited = true; }
    pdl_launch();

    // ---- computing side: the G queries as B fragments, running softmax state, O^T accumulators
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
      fire_next();
      if (!mbar_wait_bounded(bar0 + csi * 8, (phases >> csi) & 1u)) {
        // a copy did not land: flag it, give the other stages' copies their chance to land in
        // this CTA's memory while it still belongs to us, and leave the head unfinished
        if (lane == 0) atomicOr(st.errword, ERR_COPY_TIMEOUT);
        for (int s = 0; s < nst; ++s)
          if (s != csi) mbar_wait_bounded(bar0 + s * 8, (phases >> s) & 1u);
        if (local) bar_arrive(1 + first_w, 32 * npieces);   // the head's other warps must not wait for this one
        return;
      }
      phases ^= 1u << csi;
      __syncwarp();   // zero rows other lanes stored for a short group are visible
      const uint32_t stage = ring_u32 + csi * STAGE_BYTES;
      const int base = ci * GRP;
      const int valid = min(GRP, n_tot - base);
      if (p.append && ci == g_u - 1) {
        // the arriving token: its rows go from the stage into the head's spare slot
        const int e = valid - 1;
        const int slot = list[n_old];
        uint4 val;
        asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];\n" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(stage + e * ENTRY_STRIDE + lane * 16));
        *reinterpret_cast<uint4*>(st.pool + ((size_t)seq * st.slots_per_seq + slot) * SLOT_BYTES + lane * 16) = val;
        if (lane == 0) {
          st.meta_pos[mb + n_old] = p.t;
          st.meta_tau[mb + n_old] = p.t;
          st.meta_crf[mb + n_old] = 0.0f;
        }
      }
      // ---- S[key][head] = K Q^T over the 8 k-steps of 16 channels, two chains of four
      float s[4] = {0.f, 0.f, 0.f, 0.f};
      {
        float s2[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t ka = stage + kb;
#pragma unroll
        for (int ks = 0; ks < 8; ks += 2) {
          uint32_t a[4], a2[4];
          ldsm_x4(a, ka + ks * 32);
          ldsm_x4(a2, ka + ks * 32 + 32);
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
        const uint32_t va = stage + vb;
#pragma unroll
        for (int mt = 0; mt < 8; mt += 2) {   // two tiles at a time: the two MMAs of a tile depend on each other
          uint32_t a[4], a2[4];
          ldsm_x4_t(a, va + mt * 32);
          ldsm_x4_t(a2, va + mt * 32 + 32);
          mma_bf16(o[mt], a, b0, b1);
          mma_bf16(o[mt + 1], a2, b0, b1);
          mma_bf16(o[mt], a, rr0, rr1);
          mma_bf16(o[mt + 1], a2, rr0, rr1);
        }
      }
      csi = (csi + 1 == nst) ? 0 : csi + 1;
      __syncwarp();   // the stage is free for the fire of the next iteration
    }

    if (npieces == 1) {
      // ---- the whole head was this warp's: normalise and write `out` from the accumulators
      float ls0 = l0, ls1 = l1;
#pragma unroll
      for (int x = 4; x < 32; x <<= 1) {
        ls0 += __shfl_xor_sync(0xffffffffu, ls0, x);
        ls1 += __shfl_xor_sync(0xffffffffu, ls1, x);
      }
      const float i0 = 1.0f / ls0, i1 = 1.0f / ls1;
      const int h0 = 2 * tig, h1 = 2 * tig + 1;
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
      if (lane == 0) {
        atomicAdd(&st.counters[0], (unsigned long long)n_tot);
        if (!p.track) keep_and_refill(st, p.n_out, uid, seq, n_tot, p.append != 0);
      }
      continue;
    }
    if (local) {
      // ---- the piece's partial goes into this warp's ring (idle by now: every copy that was
      // fired has been consumed); after a barrier of the head's warps each of them merges a
      // share of the query heads from all the partials
      constexpr int HS = HD + 4;   // row stride that spreads the four head pairs of a store over the banks
      constexpr int WSTRIDE = STAGES * STAGE_BYTES;
      float* mine = reinterpret_cast<float*>(smem + w * WSTRIDE);
      float ls0 = l0, ls1 = l1;
#pragma unroll
      for (int x = 4; x < 32; x <<= 1) {
        ls0 += __shfl_xor_sync(0xffffffffu, ls0, x);
        ls1 += __shfl_xor_sync(0xffffffffu, ls1, x);
      }
      if (gid == 0) {
        *reinterpret_cast<float2*>(mine + 2 * tig) = make_float2(m0, m1);
        *reinterpret_cast<float2*>(mine + 8 + 2 * tig) = make_float2(ls0, ls1);
      }
      {
        const int h0 = 2 * tig, h1 = 2 * tig + 1;
        float* po = mine + 16 + gid;
#pragma unroll
        for (int mt = 0; mt < 8; ++mt) {
          if (h0 < G) { po[h0 * HS + 16 * mt] = o[mt][0]; po[h0 * HS + 16 * mt + 8] = o[mt][2]; }
          if (h1 < G) { po[h1 * HS + 16 * mt] = o[mt][1]; po[h1 * HS + 16 * mt + 8] = o[mt][3]; }
        }
      }
      bar_sync(1 + first_w, 32 * npieces);
      const unsigned char* base = smem + first_w * WSTRIDE;
      for (int g = w - first_w; g < G; g += npieces) {
        float pm[NW], pl[NW];
        float4 v[NW];
        float m = -INFINITY;
#pragma unroll
        for (int j = 0; j < NW; ++j) {
          const float* pp = reinterpret_cast<const float*>(base + (j < npieces ? j : 0) * WSTRIDE);
          pm[j] = (j < npieces) ? pp[g] : -INFINITY;
          pl[j] = (j < npieces) ? pp[8 + g] : 0.f;
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
      if (w == first_w && lane == 0) {
        atomicAdd(&st.counters[0], (unsigned long long)n_tot);
        if (!p.track) keep_and_refill(st, p.n_out, uid, seq, n_tot, p.append != 0);
      }
      continue;
    }
    // ---- publish the piece's partial and take a ticket
    float* part = p.sc.partials + ((size_t)u * p.sc.pmax + piece) * PS;
    {
      float ls0 = l0, ls1 = l1;   // l over the keys of all lanes that hold the same heads
#pragma unroll
      for (int x = 4; x < 32; x <<= 1) {
        ls0 += __shfl_xor_sync(0xffffffffu, ls0, x);
        ls1 += __shfl_xor_sync(0xffffffffu, ls1, x);
      }
      if (gid == 0) {
        *reinterpret_cast<float2*>(part + 2 * tig) = make_float2(m0, m1);
        *reinterpret_cast<float2*>(part + 8 + 2 * tig) = make_float2(ls0, ls1);
      }
      const int h0 = 2 * tig, h1 = 2 * tig + 1;
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
    // ---- merge: out = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m).  The merging warp is alone,
    // so its time is the number of dependent load rounds: loads go out in batches before anything
    // consumes them.
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
    } else if (npieces <= 8) {   // two heads x eight pieces per round
      for (int g0 = 0; g0 < G; g0 += 2) {
        float mm[2], L[2];
        float4 acc[2];
        merge_small<2, 8>(pbase, PS, npieces, g0, G, lane, mm, L, acc);
#pragma unroll
        for (int h = 0; h < 2; ++h) put(g0 + h, mm[h], L[h], acc[h]);
      }
    } else {
      const int hh = lane & 7, pl = lane >> 3;   // header phase: lane = (piece mod 4, head)
      float mm = -INFINITY, Ls = 0.f;
      for (int pc0 = 0; pc0 < npieces; pc0 += 8) {
        const int pa = pc0 + pl, pb = pc0 + pl + 4;
        const bool oa = pa < npieces, ob = pb < npieces;
        const float ma = oa ? __ldcg(pbase + (size_t)pa * PS + hh) : -INFINITY;
        const float mb_ = ob ? __ldcg(pbase + (size_t)pb * PS + hh) : -INFINITY;
        const float la = oa ? __ldcg(pbase + (size_t)pa * PS + 8 + hh) : 0.f;
        const float lb = ob ? __ldcg(pbase + (size_t)pb * PS + 8 + hh) : 0.f;
        const float mn = fmaxf(mm, fmaxf(ma, mb_));
        if (mn > -INFINITY) Ls = Ls * ex2(mm - mn) + la * ex2(ma - mn) + lb * ex2(mb_ - mn);   // ex2(-inf) = 0 covers the gaps
        mm = mn;
      }
#pragma unroll
      for (int x = 8; x < 32; x <<= 1) {   // combine the four piece classes
        const float mo = __shfl_xor_sync(0xffffffffu, mm, x), lo_ = __shfl_xor_sync(0xffffffffu, Ls, x);
        const float mn = fmaxf(mm, mo);
        if (mn > -INFINITY) Ls = Ls * ex2(mm - mn) + lo_ * ex2(mo - mn);
        mm = mn;
      }
      for (int g0 = 0; g0 < G; g0 += 2) {
        float mg[2], Lg[2];
        float4 acc[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mg[h] = __shfl_sync(0xffffffffu, mm, (g0 + h) & 7);
          Lg[h] = __shfl_sync(0xffffffffu, Ls, (g0 + h) & 7);
          acc[h] = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int pc0 = 0; pc0 < npieces; pc0 += 8) merge_rows<2, 8>(pbase, PS, npieces, pc0, g0, G, lane, mg, acc);
#pragma unroll
        for (int h = 0; h < 2; ++h) put(g0 + h, mg[h], Lg[h], acc[h]);
      }
    }
    if (lane == 0) {
      atomicAdd(&st.counters[0], (unsigned long long)n_tot);
      if (!p.track) keep_and_refill(st, p.n_out, uid, seq, n_tot, p.append != 0);
    }
  }
}

__global__ void __maxnreg__(160) attn_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const State& st = p.st;
  // Without `early` the kernel before this one may still be writing the lists this one reads.
  if (!p.early) pdl_wait();
  const int U = st.batch * st.H;
  // ring stages, then one mbarrier per stage, then the split tables
  const uint32_t bars_u32 = smem_u32(smem) + RING_BYTES;
  int* off = reinterpret_cast<int*>(smem + RING_BYTES + (NW * STAGES + NW) * 8);   // U + 1 piece prefix sums
  int* nin = off + (U + 1);                                                  // U entry counts before the step
  __shared__ int s_red[NW + 1];
  __shared__ int s_mx[NW];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;

  // This CTA's turn among the launch's CTAs, asked for now so that the answer is there when the
  // split is known (used when CTAs take whole chunks of pieces).
  // The counters of the other parity are cleared for the next launch: every take of the launch
  // before this one happened before it let this one start, and the next launch cannot start
  // before this CTA has passed the point where it lets it.
  __shared__ int s_turn;
  if (threadIdx.x == 0) {
    s_turn = atomicAdd(p.piece_ctr + 2 + p.parity, 1);
    if (blockIdx.x == 0) {
      atomicExch(p.piece_ctr + (p.parity ^ 1), 0);
      atomicExch(p.piece_ctr + 2 + (p.parity ^ 1), 0);
      __threadfence();
    }
  }
  if (threadIdx.x < NW * STAGES + NW) mbar_init(bars_u32 + threadIdx.x * 8, 1);
  asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");   // made visible to the copy engine
  // ---- every CTA derives the same split.  T = groups a piece may hold at most, chosen so that
  // the pieces of all heads fit the grid's warps: sum ceil(g_u / T) <= Gtot / T + U <= nWarps.
  const int nWarps = gridDim.x * NW;
  int T;
  {
    int mine = 0, gmax = 0;
    for (int u = tid; u < U; u += NT) {
      const int uid = ((u / st.H) * st.L + p.layer) * st.H + (u % st.H);
      int n = p.n_in[uid];
      if (p.n_limit > 0) n = min(n, p.n_limit);   // a prompt token's causal view
      nin[u] = n;
      if (u % (int)gridDim.x == (int)blockIdx.x) {   // the head's slot list is asked into L2 now (each head by one CTA): the split below takes as long as the fetch
        const char* row = reinterpret_cast<const char*>(st.list_slot + (size_t)uid * st.cap);
        for (int b = 0; b < (n + 1) * 4; b += 128) asm volatile("prefetch.global.L2 [%0];\n" ::"l"(row + b));
      }
      const int g = (n + p.append + GRP - 1) / GRP;
      mine += g;
      gmax = max(gmax, g);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) gmax = max(gmax, __shfl_xor_sync(0xffffffffu, gmax, o));
    if (lane == 0) s_mx[w] = gmax;
    int Gtot;
    block_excl_scan(mine, s_red, Gtot);   // its barriers also publish s_mx
    if (Gtot == 0) return;
    for (int x = 0; x < NW; ++x) gmax = max(gmax, s_mx[x]);
    T = (nWarps > U) ? (Gtot + (nWarps - U) - 1) / (nWarps - U) : 0x7fffffff;
    // (Pieces are not made longer than that on purpose: issuing the 16 bulk copies of a group
    // blocks the issuing warp for about half a microsecond, as long as the group's MMAs take, so
    // the copy rate of a launch grows with the number of warps that stream.)
    // Small launches would be cut into pieces of GMIN groups by the bound above.  Pieces of up to
    // PIECE_SOFT groups keep the longest unit at eight pieces, which one CTA's warps stream and merge
    // through shared memory (four pieces for units under 64 groups: shorter pieces than eight
    // groups cost more in starts than they gain in parallel streams).  Large launches are not
    // lengthened beyond that either: there every warp that does not stream costs bandwidth.
    T = max(T, min(PIECE_SOFT, gmax >= 64 ? (gmax + 7) / 8 : (gmax + 3) / 4));
    T = max(T, GMIN);
    int run = 0;
    for (int b0 = 0; b0 < U; b0 += NT) {
      const int u = b0 + tid;
      int k = 0;
      if (u < U) {
        const int g = (nin[u] + p.append + GRP - 1) / GRP;
        k = (T == 0x7fffffff) ? (g > 0) : (g + T - 1) / T;   // more heads than warps: one piece each
      }
      int tot;
      const int ex = block_excl_scan(k, s_red, tot);
      if (u < U) off[u] = run + ex;
      run += tot;
    }
    if (tid == 0) off[U] = run;
    __syncthreads();
  }
  const int Ptot = off[U];
  // Which piece a warp takes.  When every warp gets at most one, pieces go to the warps in the
  // order in which they become ready (one atomic each): CTAs that reach an SM late, because the
  // kernel ahead held it longer, then find the pieces gone instead of finishing last.
  // apc = pieces a CTA gets at most; its warps with a piece share the CTA's ring stages
  const int apc = min(NW, (Ptot + (int)gridDim.x - 1) / (int)gridDim.x);
  // A warp with four stages or more gives the last one to the slot ids of its piece (one bulk
  // copy of the list segment), so that no copy waits for a global load of ids.
  // Deep rings pay when at most two warps of a CTA stream (their few warps are then bound by
  // latency); with more, three stages and all eight warps competing for the pieces are faster.
  const int nall = apc <= 2 ? min(MAX_STAGES + 1, (NW * STAGES) / apc) : STAGES;
  const bool dyn = Ptot <= nWarps;
  if (dyn && nall > STAGES && w >= apc) return;   // a deep ring: the CTA's stages are shared out among its first apc warps
  int pi, chunk0 = -1;
  if (dyn && nall == STAGES) {
    // A CTA takes NW consecutive pieces at once, so that most heads have all their pieces in one
    // CTA and merge through shared memory.  There are at most as many such chunks as CTAs.
    chunk0 = s_turn * NW;   // written before the barriers of the split
    pi = chunk0 + w;
  } else if (dyn) {
    pi = 0;
    if (lane == 0) pi = atomicAdd(p.piece_ctr + p.parity, 1);
    pi = __shfl_sync(0xffffffffu, pi, 0);
  } else {
    pi = w * gridDim.x + blockIdx.x;   // ranks interleave over the CTAs
  }
  if (pi >= Ptot) return;

  if (nall > STAGES) stream_pieces<true>(p, smem, off, nin, U, Ptot, nWarps, nall, dyn, pi, bars_u32, -1);
  else stream_pieces<false>(p, smem, off, nin, U, Ptot, nWarps, nall, dyn, pi, bars_u32, chunk0);
}

}  // namespace ckv
