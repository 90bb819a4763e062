// Decode attention of one layer (Section 2.2): the G queries of every kv head over its
// slot-indexed cache, split-K over the warps of a persistent grid.
//
// Every warp owns a contiguous range of 16-key groups of the layer's flat group sequence
// (all heads back to back) and streams it through a private ring of shared-memory stages
// filled by 16-byte cp.async, so there is no block-wide barrier after the prologue.  Both
// contractions run on the tensor cores with keys on the MMA M dimension and the (padded)
// query heads on N = 8:   S[16 keys x 8 heads] = K Q^T,   O^T[128 x 8 heads] += V^T P^T.
// A warp publishes one (m, l, O) partial per head it touched; the warp whose partial
// completes a head merges them into `out`.  The scaled logits of the step are left in the
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

// Byte offset of 16-byte chunk `c` of row `r` inside a 16 x 256 B tile; the XOR spreads the
// eight rows an ldmatrix touches over all banks.
__device__ __forceinline__ uint32_t tile_off(int r, int c) { return (uint32_t)(r * ROW_BYTES + ((c ^ (r & 7)) << 4)); }

// One streamed group as the issuing side sees it.
struct GroupDesc {
  int u;       // head index within the launch (seq * H + kv head)
  int base;    // list position of the group's first entry
  int valid;   // entries in the group (1..16)
  int slot;    // lane e < valid: pool slot of entry base + e
};

__global__ void __launch_bounds__(NT, 1) attn_kernel(const DecodeParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const State& st = p.st;
  const int U = st.batch * st.H;
  int* off = reinterpret_cast<int*>(smem + RING_BYTES);   // U + 1 group prefix sums
  int* nin = off + (U + 1);                               // U entry counts before the step
  __shared__ int s_red[NW + 1];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int G = p.G;
  const int PS = 16 + G * HD;

  // ---- every CTA derives the same flat split of all groups of this layer
  {
    int run = 0;
    for (int b0 = 0; b0 < U; b0 += NT) {
      const int u = b0 + tid;
      int g = 0;
      if (u < U) {
        const int uid = ((u / st.H) * st.L + p.layer) * st.H + (u % st.H);
        const int n = p.n_in[uid];
        nin[u] = n;
        g = (n + p.append + GRP - 1) / GRP;
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
  const int nWarps = gridDim.x * NW;
  const int nActive = (int)min((long long)nWarps, max(1ll, Gtot / GMIN));
  const int me = w * gridDim.x + blockIdx.x;   // ranks interleave over the CTAs so small launches use every SM
  if (me >= nActive) return;
  const int lo = (int)((long long)me * Gtot / nActive), hi = (int)((long long)(me + 1) * Gtot / nActive);
  if (hi <= lo) return;
  auto rank_of = [&](int x) {   // rank of the warp whose range holds group x
    int c = (int)((long long)x * nActive / Gtot);
    while ((int)((long long)(c + 1) * Gtot / nActive) <= x) ++c;
    while ((int)((long long)c * Gtot / nActive) > x) --c;
    return c;
  };

  unsigned char* ring = smem + (size_t)w * STAGES * STAGE_BYTES;
  const uint32_t ring_u32 = smem_u32(ring);
  const int gid = lane >> 2, tig = lane & 3;
  const int mi = lane >> 3, r8 = lane & 7;
  const int chunk = lane & 15;

  // first head whose group range holds `lo`
  int u_first = 0;
  {
    int a = 0, b = U;
    while (b - a > 1) {
      const int mid = (a + b) >> 1;
      if (off[mid] <= lo) a = mid; else b = mid;
    }
    u_first = a;
  }

  // ---- issuing side
  int iu = u_first;
  auto prep = [&](int idx) {
    GroupDesc d;
    while (off[iu + 1] <= idx) ++iu;
    d.u = iu;
    d.base = (idx - off[iu]) * GRP;
    d.valid = min(GRP, nin[iu] + p.append - d.base);
    const int uid = ((iu / st.H) * st.L + p.layer) * st.H + (iu % st.H);
    d.slot = (lane < d.valid) ? st.list_slot[(size_t)uid * st.cap + d.base + lane] : 0;
    return d;
  };
  auto fire = [&](const GroupDesc& d, int stage) {
    const int seq = d.u / st.H, head = d.u % st.H;
    const unsigned char* poolseq = st.pool + (size_t)seq * st.slots_per_seq * SLOT_BYTES;
    const int n_old = nin[d.u];
    const int e_new = (p.append && n_old >= d.base && n_old < d.base + GRP) ? n_old - d.base : -1;
    const uint32_t dst0 = ring_u32 + stage * STAGE_BYTES + (lane < 16 ? 0 : GRP * ROW_BYTES);
#pragma unroll
    for (int e = 0; e < GRP; ++e) {
      const int s = __shfl_sync(0xffffffffu, d.slot, e);
      const uint32_t dst = dst0 + tile_off(e, chunk);
      if (e < d.valid) {
        const unsigned char* src = poolseq + (size_t)s * SLOT_BYTES + lane * 16;
        if (e == e_new)   // the arriving token comes from the call's inputs
          src = reinterpret_cast<const unsigned char*>((lane < 16 ? p.k_new : p.v_new) + ((size_t)seq * st.H + head) * HD) + chunk * 16;
        cp_async16(dst, src);
      } else {
        asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0) : "memory");
      }
    }
  };

  // ---- computing side: state of the head being accumulated
  int cu = -1;
  uint32_t qb[8][2];
  float o[8][4];
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  auto publish = [&]() {
    const int u = cu;
    const int seq = u / st.H, head = u % st.H;
    const int uid = (seq * st.L + p.layer) * st.H + head;
    const int g0 = off[u], g1 = off[u + 1];
    const int r_first = rank_of(g0), r_last = rank_of(g1 - 1);
    const int piece = me - r_first, npieces = r_last - r_first + 1;
    float* part = p.sc.partials + ((size_t)u * p.sc.pmax + piece) * PS;
    // l over the keys of all lanes that hold the same heads
    float ls0 = l0, ls1 = l1;
#pragma unroll
    for (int x = 4; x < 32; x <<= 1) {
      ls0 += __shfl_xor_sync(0xffffffffu, ls0, x);
      ls1 += __shfl_xor_sync(0xffffffffu, ls1, x);
    }
    if (gid == 0) {
      part[2 * tig] = m0; part[2 * tig + 1] = m1;
      part[8 + 2 * tig] = ls0; part[8 + 2 * tig + 1] = ls1;
    }
    const int h0 = 2 * tig, h1 = 2 * tig + 1;
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) {
      const int d0 = 16 * mt + gid;
      if (h0 < G) { part[16 + h0 * HD + d0] = o[mt][0]; part[16 + h0 * HD + d0 + 8] = o[mt][2]; }
      if (h1 < G) { part[16 + h1 * HD + d0] = o[mt][1]; part[16 + h1 * HD + d0 + 8] = o[mt][3]; }
    }
    __threadfence();
    __syncwarp();
    int last = 0;
    if (lane == 0) {
      const int old = atomicAdd(&p.sc.ticket[u], 1);
      last = (old == npieces - 1);
      if (last) p.sc.ticket[u] = 0;   // ready for the next launch that uses this scratch set
    }
    last = __shfl_sync(0xffffffffu, last, 0);
    if (!last) return;
    __threadfence();
    // ---- merge: out = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m), lane = 4 output channels
    const float* pbase = p.sc.partials + (size_t)u * p.sc.pmax * PS;
    const int Hq = st.H * G;
    for (int g = 0; g < G; ++g) {
      float mm = -INFINITY;
      for (int pc = 0; pc < npieces; ++pc) mm = fmaxf(mm, __ldcg(pbase + (size_t)pc * PS + g));
      float L = 0.f;
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int pc = 0; pc < npieces; ++pc) {
        const float* pp = pbase + (size_t)pc * PS;
        const float sc = ex2(__ldcg(pp + g) - mm);
        L = fmaf(__ldcg(pp + 8 + g), sc, L);
        const float4 ov = __ldcg(reinterpret_cast<const float4*>(pp + 16 + g * HD) + lane);
        acc.x = fmaf(ov.x, sc, acc.x); acc.y = fmaf(ov.y, sc, acc.y);
        acc.z = fmaf(ov.z, sc, acc.z); acc.w = fmaf(ov.w, sc, acc.w);
      }
      const float inv = 1.0f / L;
      uint2 pk;
      pk.x = pack_bf16(acc.x * inv, acc.y * inv);
      pk.y = pack_bf16(acc.z * inv, acc.w * inv);
      *reinterpret_cast<uint2*>(p.out + ((size_t)seq * Hq + head * G + g) * HD + lane * 4) = pk;
      if (lane == 0 && p.track) p.sc.mfin[u * QH + g] = mm;
    }
    if (lane == 0) {
      const int n_tot = nin[u] + p.append;
      atomicAdd(&st.counters[0], (unsigned long long)n_tot);
      if (!p.track) keep_and_refill(st, p.n_out, uid, seq, n_tot, p.append != 0);
    }
  };

  auto enter = [&](int idx) {   // start accumulating the head that holds group idx
    cu = (cu < 0) ? u_first : cu + 1;
    while (off[cu + 1] <= idx) ++cu;
    const int seq = cu / st.H, head = cu % st.H;
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q + ((size_t)seq * st.H * G + head * G + gid) * HD);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qb[ks][0] = (gid < G) ? q32[ks * 8 + tig] : 0u;
      qb[ks][1] = (gid < G) ? q32[ks * 8 + tig + 4] : 0u;
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }
    m0 = -INFINITY; m1 = -INFINITY; l0 = 0.f; l1 = 0.f;
  };

  auto compute = [&](int idx, int stage) {
    const int u = cu;
    const int base = (idx - off[u]) * GRP;
    const int n_old = nin[u], n_tot = n_old + p.append;
    const int valid = min(GRP, n_tot - base);
    const uint32_t sK = ring_u32 + stage * STAGE_BYTES, sV = sK + GRP * ROW_BYTES;
    if (p.append && n_old >= base && n_old < base + GRP) {
      // the arriving token: its rows go from the stage into the head's spare slot
      const int seq = u / st.H;
      const int uid = (seq * st.L + p.layer) * st.H + (u % st.H);
      const size_t mb = (size_t)uid * st.cap;
      const int e = n_old - base;
      const int slot = st.list_slot[mb + n_old];
      uint4 val;
      const uint32_t src = (lane < 16 ? sK : sV) + tile_off(e, chunk);
      asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];\n" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(src));
      *reinterpret_cast<uint4*>(st.pool + ((size_t)seq * st.slots_per_seq + slot) * SLOT_BYTES + lane * 16) = val;
      if (lane == 0) {
        st.meta_pos[mb + n_old] = p.t;
        st.meta_tau[mb + n_old] = p.t;
        st.meta_crf[mb + n_old] = 0.0f;
      }
    }
    // ---- S[key][head] = K Q^T over the 8 k-steps of 16 channels
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const int krow = (mi & 1) * 8 + r8;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t a[4];
        ldsm_x4(a, sK + tile_off(krow, 2 * ks + (mi >> 1)));
        mma_bf16(s, a, qb[ks][0], qb[ks][1]);
      }
    }
    const bool v0 = gid < valid, v1 = gid + 8 < valid;
    if (p.track) {
      float* lrow = p.sc.logits + ((size_t)u * p.sc.cap_s + base) * QH + 2 * tig;
      if (v0) *reinterpret_cast<float2*>(lrow + (size_t)gid * QH) = make_float2(__fmul_rn(s[0], p.scale), __fmul_rn(s[1], p.scale));
      if (v1) *reinterpret_cast<float2*>(lrow + (size_t)(gid + 8) * QH) = make_float2(__fmul_rn(s[2], p.scale), __fmul_rn(s[3], p.scale));
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
    const float n0 = fmaxf(m0, c0), n1 = fmaxf(m1, c1);
    if (__any_sync(0xffffffffu, n0 > m0 || n1 > m1)) {
      const float r0 = ex2(m0 - n0), r1 = ex2(m1 - n1);
      l0 *= r0; l1 *= r1;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) { o[mt][0] *= r0; o[mt][1] *= r1; o[mt][2] *= r0; o[mt][3] *= r1; }
      m0 = n0; m1 = n1;
    }
    const float p0 = ex2(t0 - m0), p1 = ex2(t1 - m1), p2 = ex2(t2 - m0), p3 = ex2(t3 - m1);
    l0 += p0 + p2;
    l1 += p1 + p3;
    // P^T as the B operand: transpose the two 8 x 8 (key x head) blocks across the warp
    const uint32_t b0 = movm_t(pack_bf16(p0, p1)), b1 = movm_t(pack_bf16(p2, p3));
    // ---- O^T[channel][head] += V^T P^T, 8 tiles of 16 channels
    {
      const int vrow = (mi >> 1) * 8 + r8;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        uint32_t a[4];
        ldsm_x4_t(a, sV + tile_off(vrow, 2 * mt + (mi & 1)));
        mma_bf16(o[mt], a, b0, b1);
      }
    }
  };

  // ---- the pipeline: groups lo .. hi-1 flow through the ring, STAGES-1 of them in flight
  GroupDesc nd = prep(lo);
  int next = lo;   // next group to fire
#pragma unroll 1
  for (int s = 0; s < STAGES - 1; ++s) {
    if (next < hi) {
      const GroupDesc d = nd;
      ++next;
      if (next < hi) nd = prep(next);
      fire(d, s);
    }
    cp_commit();
  }
#pragma unroll 1
  for (int ci = lo; ci < hi; ++ci) {
    const int k = ci - lo;
    if (next < hi) {
      const GroupDesc d = nd;
      ++next;
      if (next < hi) nd = prep(next);
      fire(d, (k + STAGES - 1) % STAGES);
    }
    cp_commit();
    cp_wait<STAGES - 1>();
    __syncwarp();
    if (cu < 0 || ci >= off[cu + 1]) {
      if (cu >= 0) publish();
      enter(ci);
    }
    compute(ci, k % STAGES);
    __syncwarp();   // the stage is free for the fire of the next iteration
  }
  publish();
}

}  // namespace ckv
