// Shared definitions of the Crystal-KV CUDA path (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ckv {

constexpr int HD = 128;             // head_dim
constexpr int ROW_BYTES = 256;      // one K or V row, bf16
constexpr int SLOT_BYTES = 512;     // pool slot = K row followed by V row
constexpr int GRP = 16;             // keys per streamed group (one MMA tile of keys)
constexpr int NW = 8;               // warps per CTA
constexpr int NT = NW * 32;
constexpr int STAGES = 3;           // ring depth per warp, in groups
constexpr int STAGE_BYTES = GRP * (SLOT_BYTES + 16);   // 16 entries, each K row + V row + 16 B of padding
constexpr int RING_BYTES = NW * STAGES * STAGE_BYTES;  // 198 KB
constexpr int GMIN = 4;             // fewest groups a working warp takes
constexpr int QH = 8;               // query heads of a group as padded for the MMA N dimension
constexpr int MAX_UNITS_PER_CALL = 2048;   // bounded by the split tables in shared memory
constexpr int NSETS = 16;           // logit scratch sets cycled by consecutive tracked launches

// error word bits raised by device-side consistency checks (never a trap)
constexpr int ERR_FREE_UNDERFLOW = 1;   // a head needed a slot and the sequence's free list was empty
constexpr int ERR_OVER_EVICT = 2;       // a decode step found a head further over its budget than the eviction period allows
constexpr int ERR_CAPACITY = 4;         // a head's list would outgrow its capacity
constexpr int ERR_NUCLEUS = 8;          // the top-p threshold search did not find its boundary
constexpr int ERR_COPY_TIMEOUT = 16;    // a bulk copy into shared memory did not complete within a second

struct State {
  // K/V pool: [batch][slots_per_seq][512 B]
  unsigned char* pool;
  long long slots_per_seq;
  int* free_stack;   // [batch][slots_per_seq]
  int* free_top;     // [batch] number of free slots
  // per unit (uid = (seq*L + layer)*H + head), capacity `cap` list positions
  int* list_slot;    // [units][cap] slot of the entry at a list position; position n holds the spare
  int* meta_pos;     // [units][cap] token position
  int* meta_tau;     // [units][cap] last hit time
  float* meta_crf;   // [units][cap] CRF at tau
  int* nbuf[2];      // [2][units] entry counts, double buffered: a step reads one and writes the other
  int* budget;       // [units] == [batch][L][H]
  int* own;          // [units] list positions [0, own) hold slots that belong to the head: its entries, then
                     // its spares (one in steady state; up to the eviction period with a buffered cadence)
  const float* tab;  // lambda^D, D in [0, max_context]
  int* errword;
  unsigned long long* counters;  // entries attended, hits, evictions
  int batch, L, H, cap;
};

// scratch of one launch pair (attention kernel, then LRFU kernel), assembled per launch: the
// logits and (m, l) come from one of NSETS cycled sets, the partials and tickets from one of two
struct Scratch {
  float* logits;     // [U][cap_s][QH] scaled logits of the step, one 32-byte row per entry
  float* pbar;       // [U][cap_s] group-mean probabilities (reused as int scratch)
  float* partials;   // [U][pmax][16 + G*128] split-K partial: m[8], l[8], O[G][128]
  float* mfin;       // [U][2][QH] per query head: merged reference point (log2 domain), then normaliser
  int* ticket;       // [U]
  int cap_s, pmax;
};

struct DecodeParams {
  State st;
  Scratch sc;
  const __nv_bfloat16* q;       // [batch][Hq][128]
  const __nv_bfloat16* k_new;   // [batch][H][128]
  const __nv_bfloat16* v_new;
  __nv_bfloat16* out;           // [batch][Hq][128]
  int* piece_ctr;    // counters by launch parity: [0..1] the attention warps take pieces, [2..3] its CTAs take chunks of pieces
  int parity;
  const int* n_in;   // entry counts before this step
  int* n_out;        // entry counts after it
  int layer;
  int G;          // query heads per kv head
  int t;          // time of this step
  int append;     // 1: decode (a new entry arrives); 0: scoring pass over the prompt
  int track;      // 1: Algorithm 1 runs (hits, CRF, eviction) in the LRFU kernel that follows
  int release;    // 1: freed slots beyond one spare go back to the free list (no pops in this launch)
  int early;      // 1: the lists and rows of this layer are final, so the attention kernel may read them
                  //    before the kernel ahead of it in the stream has completed
  int n_limit;    // > 0: only the first n_limit entries of every head take part (a prompt token's causal view)
  int hold;       // 1: Algorithm 1 stops after step 3; lengths and lists stay as they are
  int evict_every;   // m >= 1: step 4 waits until a head is m entries over its budget, then removes them all
  int literal;    // 1: Algorithm 1 is skipped for a head below its budget (its first line as printed)
  float scale;    // logit scale
  float scale_log2;
  float top_p;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() {
  asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory");
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

// A head keeps its length and, unless it still owns a spare there, takes a fresh slot for list
// position n (decode steps in which nothing left the head).  One thread calls it.
__device__ __forceinline__ void keep_and_refill(const State& st, int* n_out, int uid, int seq, int n,
                                                bool append) {
  n_out[uid] = n;
  if (!append) return;
  if (st.own[uid] > n) return;   // one of the head's own spares is at list position n already
  if (n + 1 > st.cap) {
    atomicOr(st.errword, ERR_CAPACITY);
    return;
  }
  const int idx = atomicSub(&st.free_top[seq], 1) - 1;
  if (idx < 0) {
    atomicAdd(&st.free_top[seq], 1);
    atomicOr(st.errword, ERR_FREE_UNDERFLOW);
  } else {
    st.list_slot[(size_t)uid * st.cap + n] = st.free_stack[(size_t)seq * st.slots_per_seq + idx];
    st.own[uid] = n + 1;
  }
}

}  // namespace ckv
