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

// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start while the kernel before it in the stream still runs; pdl_wait() returns once that
// kernel has completed and its writes are visible, pdl_launch() lets the kernel after this
// one start.  Both are no-ops for a launch without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;\n" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;\n" ::: "memory"); }

// Byte offset of 16-byte chunk `c` of row `r` inside a 16 x 256 B tile; the XOR spreads the
// eight rows an ldmatrix touches over all banks.
__device__ __forceinline__ uint32_t tile_off(int r, int c) { return (uint32_t)(r * ROW_BYTES + ((c ^ (r & 7)) << 4)); }

// One streamed group as the issuing side sees it.
struct GroupDesc {
  int u;       // head index within the launch (seq * H + kv head)
  int valid;   // entries in the group (1..16)
  int has_new; // the group's last entry is the arriving token
  int slot;    // lane e < valid: pool slot of entry base + e
  const unsigned char* pool;   // the sequence's pool, advanced to this lane's 16-byte chunk
};

constexpr float LAZY = 8.0f;   // the running maximum (log2 domain) may trail the true one by this much

__global__ void __launch_bounds__(NT, 1) attn_kernel(const DecodeParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const State& st = p.st;
  // Without `early` the kernel before this one may still be writing the lists this one reads.
  if (!p.early) pdl_wait();
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
  const unsigned Gtot = (unsigned)off[U];
  if (Gtot == 0) return;
  const unsigned nWarps = gridDim.x * NW;
  const unsigned per = max((unsigned)GMIN, (Gtot + nWarps - 1) / nWarps);   // groups per working warp
  const unsigned me = w * gridDim.x + blockIdx.x;   // ranks interleave over the CTAs so small launches use every SM
  if ((unsigned long long)me * per >= Gtot) return;
  const int lo = (int)(me * per), hi = (int)min(me * per + per, Gtot);

  const uint32_t ring_u32 = smem_u32(smem) + w * (STAGES * STAGE_BYTES);
  const int gid = lane >> 2, tig = lane & 3;
  const int mi = lane >> 3, r8 = lane & 7;
  const int chunk = lane & 15;
  const uint32_t half_off = lane < 16 ? 0u : (uint32_t)(GRP * ROW_BYTES);
  // cp.async destination of this lane's chunk in row e of a stage: xoff[e & 7] + e * 256
  uint32_t xoff[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) xoff[j] = half_off + (uint32_t)((chunk ^ j) << 4);
  // ldmatrix row addresses: K tile of k-step ks at (stage + kb) ^ (ks << 5), V tile of channel
  // tile mt at (stage + vb) ^ (mt << 5); stages are 256-byte aligned so the XOR is carry free
  const uint32_t kb = (uint32_t)(((mi & 1) * 8 + r8) * ROW_BYTES + (((mi >> 1) ^ r8) << 4));
  const uint32_t vb = (uint32_t)(GRP * ROW_BYTES + ((mi >> 1) * 8 + r8) * ROW_BYTES + (((mi & 1) ^ r8) << 4));
  const unsigned char* newrow_lane =
      reinterpret_cast<const unsigned char*>(lane < 16 ? p.k_new : p.v_new) + chunk * 16;

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

  // ---- issuing side: registers of the head whose groups are being requested
  int iu = u_first, i_seq = u_first / st.H, i_head = u_first % st.H;
  int i_off, i_end, i_ntot;
  const int* i_list;
  const unsigned char* i_pool;
  auto issue_unit = [&]() {
    i_off = off[iu];
    i_end = off[iu + 1];
    i_ntot = nin[iu] + p.append;
    const int uid = (i_seq * st.L + p.layer) * st.H + i_head;
    i_list = st.list_slot + (size_t)uid * st.cap;
    i_pool = st.pool + (size_t)i_seq * st.slots_per_seq * SLOT_BYTES + lane * 16;
  };
  issue_unit();
  auto prep = [&](int idx) {
    if (idx >= i_end) {
      do {
        ++iu;
        if (++i_head == st.H) { i_head = 0; ++i_seq; }
      } while (off[iu + 1] <= idx);
      issue_unit();
    }
    GroupDesc d;
    const int base = (idx - i_off) * GRP;
    d.u = iu;
    d.valid = min(GRP, i_ntot - base);
    d.has_new = p.append && (base + d.valid == i_ntot);
    d.slot = (lane < d.valid) ? i_list[base + lane] : 0;
    d.pool = i_pool;
    return d;
  };
  auto fire = [&](const GroupDesc& d, uint32_t stage) {
    if (d.valid == GRP && !d.has_new) {
#pragma unroll
      for (int e = 0; e < GRP; ++e) {
        const unsigned s = (unsigned)__shfl_sync(0xffffffffu, d.slot, e);
        cp_async16(stage + xoff[e & 7] + e * ROW_BYTES, d.pool + (size_t)s * SLOT_BYTES);
      }
    } else {
      const int nv = d.valid - d.has_new;   // entries that come from the pool
#pragma unroll
      for (int e = 0; e < GRP; ++e) {
        const unsigned s = (unsigned)__shfl_sync(0xffffffffu, d.slot, e);
        const uint32_t dst = stage + xoff[e & 7] + e * ROW_BYTES;
        if (e < nv) {
          cp_async16(dst, d.pool + (size_t)s * SLOT_BYTES);
        } else if (e >= d.valid) {
          asm volatile("st.shared.v4.b32 [%0], {%1,%1,%1,%1};\n" ::"r"(dst), "r"(0) : "memory");
        }
      }
      if (d.has_new) {   // the arriving token comes from the call's inputs
        pdl_wait();
        const int e = d.valid - 1;
        cp_async16(stage + half_off + tile_off(e, chunk), newrow_lane + (size_t)d.u * ROW_BYTES);
      }
    }
  };

  // ---- computing side: state of the head being accumulated
  int cu = -1, c_seq = 0, c_head = 0, c_off = 0, c_end = 0, c_nold = 0;
  float* c_logit = nullptr;
  uint32_t qb[8][2];
  float o[8][4];
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

  auto publish = [&]() {
    const int u = cu;
    const int uid = (c_seq * st.L + p.layer) * st.H + c_head;
    const unsigned r_first = (unsigned)c_off / per, r_last = (unsigned)(c_end - 1) / per;
    const int piece = (int)(me - r_first), npieces = (int)(r_last - r_first + 1);
    float* part = p.sc.partials + ((size_t)u * p.sc.pmax + piece) * PS;
    // l over the keys of all lanes that hold the same heads
    float ls0 = l0, ls1 = l1;
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
    // ---- merge: out = sum_p O_p 2^(m_p - m) / sum_p l_p 2^(m_p - m).  Loads that do not depend
    // on one another are issued together: first every piece's (m, l) header, then the O rows.
    const float* pbase = p.sc.partials + (size_t)u * p.sc.pmax * PS;
    const int Hq = st.H * G;
    const int hh = lane & 7, pl = lane >> 3;   // header phase: lane = (piece mod 4, head)
    float mm = -INFINITY;
    for (int pc = pl; pc < npieces; pc += 4) mm = fmaxf(mm, __ldcg(pbase + (size_t)pc * PS + hh));
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, 8));
    mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, 16));
    float Ls = 0.f;
    for (int pc = pl; pc < npieces; pc += 4)
      Ls = fmaf(__ldcg(pbase + (size_t)pc * PS + 8 + hh), ex2(__ldcg(pbase + (size_t)pc * PS + hh) - mm), Ls);
    Ls += __shfl_xor_sync(0xffffffffu, Ls, 8);
    Ls += __shfl_xor_sync(0xffffffffu, Ls, 16);
    if (lane < G && p.track) {   // reference point and normaliser of the step's softmax, for the LRFU kernel
      p.sc.mfin[u * (2 * QH) + lane] = mm;
      p.sc.mfin[u * (2 * QH) + QH + lane] = Ls;
    }
    float mg[QH], inv[QH];
#pragma unroll
    for (int g = 0; g < QH; ++g) {
      mg[g] = __shfl_sync(0xffffffffu, mm, g);
      inv[g] = 1.0f / __shfl_sync(0xffffffffu, Ls, g);
    }
    float4 acc[QH];   // lane = 4 output channels of every head
#pragma unroll
    for (int g = 0; g < QH; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int pc = 0; pc < npieces; ++pc) {
      const float* pp = pbase + (size_t)pc * PS;
#pragma unroll
      for (int g = 0; g < QH; ++g) {
        if (g < G) {
          const float sc = ex2(__ldcg(pp + g) - mg[g]);
          const float4 ov = __ldcg(reinterpret_cast<const float4*>(pp + 16 + g * HD) + lane);
          acc[g].x = fmaf(ov.x, sc, acc[g].x); acc[g].y = fmaf(ov.y, sc, acc[g].y);
          acc[g].z = fmaf(ov.z, sc, acc[g].z); acc[g].w = fmaf(ov.w, sc, acc[g].w);
        }
      }
    }
#pragma unroll
    for (int g = 0; g < QH; ++g) {
      if (g < G) {
        uint2 pk;
        pk.x = pack_bf16(acc[g].x * inv[g], acc[g].y * inv[g]);
        pk.y = pack_bf16(acc[g].z * inv[g], acc[g].w * inv[g]);
        *reinterpret_cast<uint2*>(p.out + ((size_t)(u * G + g)) * HD + lane * 4) = pk;
      }
    }
    (void)Hq;
    if (lane == 0) {
      const int n_tot = c_nold + p.append;
      atomicAdd(&st.counters[0], (unsigned long long)n_tot);
      if (!p.track) keep_and_refill(st, p.n_out, uid, c_seq, n_tot, p.append != 0);
    }
  };

  auto enter = [&](int idx) {   // start accumulating the head that holds group idx
    if (cu < 0) {
      cu = u_first; c_seq = u_first / st.H; c_head = u_first % st.H;
    } else {
      do {
        ++cu;
        if (++c_head == st.H) { c_head = 0; ++c_seq; }
      } while (off[cu + 1] <= idx);
    }
    c_off = off[cu];
    c_end = off[cu + 1];
    c_nold = nin[cu];
    c_logit = p.sc.logits + (size_t)cu * p.sc.cap_s * QH + gid * QH + 2 * tig;
    const uint32_t* q32 = reinterpret_cast<const uint32_t*>(p.q + ((size_t)cu * G + gid) * HD);
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qb[ks][0] = (gid < G) ? q32[ks * 8 + tig] : 0u;
      qb[ks][1] = (gid < G) ? q32[ks * 8 + tig + 4] : 0u;
    }
#pragma unroll
    for (int mt = 0; mt < 8; ++mt) { o[mt][0] = 0.f; o[mt][1] = 0.f; o[mt][2] = 0.f; o[mt][3] = 0.f; }
    m0 = -INFINITY; m1 = -INFINITY; l0 = 0.f; l1 = 0.f;
  };

  auto compute = [&](int idx, uint32_t stage) {
    const int base = (idx - c_off) * GRP;
    const int n_tot = c_nold + p.append;
    const int valid = min(GRP, n_tot - base);
    if (p.append && base + valid == n_tot) {
      // the arriving token: its rows go from the stage into the head's spare slot
      const int uid = (c_seq * st.L + p.layer) * st.H + c_head;
      const size_t mb = (size_t)uid * st.cap;
      const int e = valid - 1;
      const int slot = st.list_slot[mb + c_nold];
      uint4 val;
      const uint32_t src = stage + half_off + tile_off(e, chunk);
      asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];\n" : "=r"(val.x), "=r"(val.y), "=r"(val.z), "=r"(val.w) : "r"(src));
      *reinterpret_cast<uint4*>(st.pool + ((size_t)c_seq * st.slots_per_seq + slot) * SLOT_BYTES + lane * 16) = val;
      if (lane == 0) {
        st.meta_pos[mb + c_nold] = p.t;
        st.meta_tau[mb + c_nold] = p.t;
        st.meta_crf[mb + c_nold] = 0.0f;
      }
    }
    // ---- S[key][head] = K Q^T over the 8 k-steps of 16 channels
    float s[4] = {0.f, 0.f, 0.f, 0.f};
    {
      const uint32_t ka = stage + kb;
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t a[4];
        ldsm_x4(a, ka ^ (uint32_t)(ks << 5));
        mma_bf16(s, a, qb[ks][0], qb[ks][1]);
      }
    }
    const bool v0 = gid < valid, v1 = gid + 8 < valid;
    if (p.track) {
      float* lrow = c_logit + (size_t)base * QH;
      if (v0) *reinterpret_cast<float2*>(lrow) = make_float2(__fmul_rn(s[0], p.scale), __fmul_rn(s[1], p.scale));
      if (v1) *reinterpret_cast<float2*>(lrow + 8 * QH) = make_float2(__fmul_rn(s[2], p.scale), __fmul_rn(s[3], p.scale));
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
    const uint32_t r0 = movm_t(pack_bf16(p0 - __low2float(h01), p1 - __high2float(h01)));
    const uint32_t r1 = movm_t(pack_bf16(p2 - __low2float(h23), p3 - __high2float(h23)));
    // ---- O^T[channel][head] += V^T P^T, 8 tiles of 16 channels
    {
      const uint32_t va = stage + vb;
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        uint32_t a[4];
        ldsm_x4_t(a, va ^ (uint32_t)(mt << 5));
        mma_bf16(o[mt], a, b0, b1);
        mma_bf16(o[mt], a, r0, r1);
      }
    }
  };

  // ---- the pipeline: groups lo .. hi-1 flow through the ring, STAGES-1 of them in flight; the
  // slot ids of a group are requested two fires before they are needed
  GroupDesc nd0 = prep(lo), nd1 = nd0;
  if (lo + 1 < hi) nd1 = prep(lo + 1);
  int next = lo;   // next group to fire
  uint32_t fs = ring_u32;   // stage the next fire fills
  auto fire_next = [&]() {
    if (next < hi) {
      const GroupDesc d = nd0;
      nd0 = nd1;
      if (next + 2 < hi) nd1 = prep(next + 2);
      ++next;
      fire(d, fs);
    }
    cp_commit();
    fs += STAGE_BYTES;
  };
  const uint32_t ring_end = ring_u32 + STAGES * STAGE_BYTES;
#pragma unroll 1
  for (int s = 0; s < STAGES - 1; ++s) fire_next();
  // everything above reads only the cache and its lists; the call's inputs (q, the arriving
  // row is fetched by the cp.async of a head's last group) may come from the kernel before
  pdl_wait();
  pdl_launch();
  uint32_t cs = ring_u32;   // stage the next compute reads
#pragma unroll 1
  for (int ci = lo; ci < hi; ++ci) {
    fire_next();
    if (fs == ring_end) fs = ring_u32;
    cp_wait<STAGES - 1>();
    __syncwarp();
    if (ci >= c_end) {
      if (cu >= 0) publish();
      enter(ci);
    }
    compute(ci, cs);
    cs += STAGE_BYTES;
    if (cs == ring_end) cs = ring_u32;
    __syncwarp();   // the stage is free for the fire of the next iteration
  }
  publish();
}

}  // namespace ckv
