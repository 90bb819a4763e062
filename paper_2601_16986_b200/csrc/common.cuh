// Shared definitions of the Crystal-KV CUDA path (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ckv {

constexpr int HD = 128;             // head_dim
constexpr int ROW_BYTES = 256;      // one K or V row, bf16
constexpr int SLOT_BYTES = 512;     // one entry in the pool: K row followed by V row
constexpr int GRP = 16;             // entries per page = keys per streamed group (one MMA tile of keys)
constexpr int PAGE_BYTES = GRP * SLOT_BYTES;   // 8 KB: what one bulk copy brings into a ring stage
constexpr int NW = 8;               // warps per CTA
constexpr int NT = NW * 32;
constexpr int STAGES = 3;           // ring depth per warp, in pages
constexpr int RING_BYTES = NW * STAGES * PAGE_BYTES;   // 192 KB
constexpr int GMIN = 4;             // fewest groups a streaming warp is given
constexpr int GLAT = 12;            // ... raised up to this many to keep a head's pieces within the eight warps of one CTA
constexpr int QH = 8;               // query heads of a group as padded for the MMA N dimension
constexpr int MAX_UNITS_PER_CALL = 2048;   // heads of one layer launch (bounded by the planner's shared memory)
constexpr int NSETS = 16;           // logit scratch sets cycled by consecutive launches
constexpr int FIFO = 8;             // pieces a warp may have fetched ahead of the one it computes (> STAGES)

// error word bits raised by device-side consistency checks (never a trap)
constexpr int ERR_FREE_UNDERFLOW = 1;   // a head needed a page and the sequence's free list was empty
constexpr int ERR_OVER_EVICT = 2;       // a decode step found a head further over its budget than the eviction period allows
constexpr int ERR_CAPACITY = 4;         // a head's list would outgrow its capacity
constexpr int ERR_NUCLEUS = 8;          // the top-p threshold search did not find its boundary
constexpr int ERR_COPY_TIMEOUT = 16;    // a bulk copy into shared memory did not complete within a second
constexpr int ERR_PLAN = 32;            // the launch plan of a layer does not match the grid it is used with

// Layout of a pool page: entry e (0..15) occupies bytes [512 e, 512 e + 512): its K row, then its
// V row, as 32 chunks of 16 bytes; chunk c is stored at chunk index c ^ (e & 7).  A page copied
// as it is into shared memory can then be read by ldmatrix (eight entries, one chunk column)
// without bank conflicts, and one bulk copy brings a whole group of keys.
__host__ __device__ __forceinline__ int chunk_offset(int e, int c) { return e * SLOT_BYTES + ((c ^ (e & 7)) << 4); }

struct State {
  // K/V pool: [batch][pages_per_seq][8192 B]
  unsigned char* pool;
  long long pages_per_seq;
  int* free_stack;   // [batch][pages_per_seq] free page ids of a sequence
  int* free_top;     // [batch] number of free pages
  // per unit (uid = (seq*L + layer)*H + head): `cap` list positions, page j backs positions 16 j .. 16 j + 15
  int* ptab;         // [units][capg] page id per 16 list positions; the first npages are owned by the unit
  int* meta_pos;     // [units][cap] token position
  int* meta_tau;     // [units][cap] last hit time
  float* meta_crf;   // [units][cap] CRF at tau
  int* n_cur;        // [units] live entries
  int* hole;         // [units] list position the next arriving entry is written to (<= n).  The live entries
                     // are the positions 0 .. n without the hole (hole == n: positions 0 .. n-1).  An entry that
                     // leaves in a decode step leaves its place to the next arrival: nothing is moved.
  int* npages;       // [units] pages owned; 16 * npages > n always (the hole is backed)
  int* budget;       // [units] == [batch][L][H]
  const float* tab;  // lambda^D, D in [0, max_context]
  int* errword;
  unsigned long long* counters;  // entries attended, hits, evictions
  int batch, L, H, cap, capg;
};

// Launch plan of one layer, read by its next attention launch: every head cut into k pieces of
// nearly equal length, one piece per streaming warp (plan.cuh).  A piece is named by (head, j, k)
// and covers groups [g j / k, g (j + 1) / k) of the head's g groups AT LAUNCH TIME, so a plan stays
// correct when heads grow or shrink by a few entries; it is rewritten when a head's group count has
// drifted from the one it was made for by an eighth (at least two), and after every reallocation.
struct Plan {
  int4* desc;        // [pd_cap] pieces, head after head: {head index u, piece j, pieces k of the head, how they are placed}
  int4* wrange;      // [warps] pieces [x, y) of the physical warp cta * NW + w; z, w: the descriptor of piece x
                     // packed (z = head index, w = j | k << 12 | placement << 24) so that a warp starts without
                     // a second dependent read, or z = -1: read desc[x]
  int* npc;          // [U] pieces per head
  int* gplan;        // [U] groups per head the plan was made for
  int* hdr;          // [4] pieces in total, groups in total, warps the plan was made for, append it was made for
};

// scratch of one launch pair (attention kernel, then LRFU kernel), assembled per launch: the
// logits and (m, l) come from one of NSETS cycled sets, the partials and tickets from one of two
struct Scratch {
  float* logits;     // [U][cap_s][QH] scaled logits of the step, one 32-byte row per list position
  float* pbar;       // [U][cap_s] group-mean probabilities (reused as int scratch)
  float* partials;   // [U][pmax][16 + G*128] split-K partial: m[8], l[8], O[G][128]
  float* mfin;       // [U][2][QH] per query head: merged reference point (log2 domain), then normaliser
  int* ticket;       // [U]
  int cap_s, pmax;
};

struct DecodeParams {
  State st;
  Scratch sc;
  Plan plan;                    // of this layer
  const __nv_bfloat16* q;       // [batch][Hq][128]
  const __nv_bfloat16* k_new;   // [batch][H][128]
  const __nv_bfloat16* v_new;
  __nv_bfloat16* out;           // [batch][Hq][128]
  int* done_ctr;     // LRFU kernel: [0] counts its finished CTAs, [1] set when a head's group count changed: the
                     // last CTA then writes the layer's next plan
  int layer;
  int G;          // query heads per kv head
  int t;          // time of this step
  int append;     // 1: decode (a new entry arrives); 0: scoring pass over the prompt
  int track;      // 1: Algorithm 1 runs (hits, CRF, eviction) in the LRFU kernel that follows
  int release;    // 1: pages a head no longer needs go back to the free list (no pops in this launch)
  int early;      // 1: the lists and rows of this layer are final, so the attention kernel may read them
                  //    before the kernel ahead of it in the stream has completed
  int n_limit;    // > 0: only the first n_limit entries of every head take part (a prompt token's causal view)
  int hold;       // 1: Algorithm 1 stops after step 3; lengths and lists stay as they are
  int evict_every;   // m >= 1: step 4 waits until a head is m entries over its budget, then removes them all
  int literal;    // 1: Algorithm 1 is skipped for a head below its budget (its first line as printed)
  int rows_absent;   // 1: the heads' entries are only metadata so far (a prompt being scored before its
                     //    survivors' rows are stored): nothing touches pool pages
  int plan_append;   // what the plan the LRFU kernel leaves behind is for: 1 = a decode step, 0 = a scoring pass
  int plan_warps;    // warps of the attention grid the plan is made for
  int plan_grid;     // CTAs of that grid
  float scale;    // logit scale
  float scale_log2;
  float top_p;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// ---- block-wide helpers (NT threads) ----
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ int warp_sum_i(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Exclusive scan of one int per thread across the block; returns this thread's prefix and
// the block total.  `red` needs NW+1 ints.  Contains two __syncthreads().
__device__ __forceinline__ int block_excl_scan(int v, int* red, int& total) {
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int x = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += x;
  }
  __syncthreads();
  if (lane == 31) red[w] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int i = 0; i < NW; ++i) {
    int x = red[i];
    if (i < w) base += x;
    tot += x;
  }
  total = tot;
  return base + inc - v;
}

// Address of chunk c (16 bytes) of the entry at list position i of a head.
__device__ __forceinline__ unsigned char* entry_chunk(const State& st, int uid, int seq, int i, int c) {
  const int page = st.ptab[(size_t)uid * st.capg + (i >> 4)];
  return st.pool + ((size_t)seq * st.pages_per_seq + page) * PAGE_BYTES + chunk_offset(i & (GRP - 1), c);
}

// Makes sure list position `need` of a head is backed by a page (a head that grew past its last
// page takes one from its sequence's free list).  One thread calls it; launches in which heads
// return pages never call it.
__device__ __forceinline__ void back_position(const State& st, int uid, int seq, int need) {
  const int have = st.npages[uid];
  if (need < have * GRP) return;
  if (need >= st.cap) {
    atomicOr(st.errword, ERR_CAPACITY);
    return;
  }
  const int idx = atomicSub(&st.free_top[seq], 1) - 1;
  if (idx < 0) {
    atomicAdd(&st.free_top[seq], 1);
    atomicOr(st.errword, ERR_FREE_UNDERFLOW);
  } else {
    st.ptab[(size_t)uid * st.capg + have] = st.free_stack[(size_t)seq * st.pages_per_seq + idx];
    st.npages[uid] = have + 1;
  }
}

// A head keeps all n entries of a step: the next arrival goes behind them.
__device__ __forceinline__ void keep_all(const State& st, int uid, int seq, int n, bool will_append) {
  st.n_cur[uid] = n;
  st.hole[uid] = n;
  if (will_append) back_position(st, uid, seq, n);
}

// List position of the i-th live entry of a head (i in [0, n)) given its hole.
__device__ __forceinline__ int live_pos(int i, int hole) { return i + (i >= hole ? 1 : 0); }

}  // namespace ckv
