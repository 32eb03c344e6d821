// The two device stages of one TOVA decode step (sm_100a).
//
//   split kernel    : one warp streams the cached K/V rows of one (sequence, KV
//                     head, chunk of rows) through a private shared-memory ring
//                     fed by bulk asynchronous copies, computes the logits of
//                     the query heads that share the KV head (Eq. 4), keeps an
//                     online soft-max (max, sum, weighted V sum) per head: the
//                     chunk's partial (Eq. 7); every logit is kept in an fp32
//                     scratch.  When the state splits into few chunks, the
//                     warps of a head group run as one CTA (or a cluster of
//                     CTAs), merge their partials in shared memory and write
//                     the attention output themselves; otherwise each warp is
//                     its own CTA and the partials go through global memory.
//   combine kernel  : merges the partials into the attention output where the
//                     split kernel has not, forms the head-averaged weights
//                     from the kept logits, takes the arg-min and overwrites
//                     the victim's row with the new token (Section 4, Eq. 9,
//                     Algorithm 1).  The Window and "+i" policies of Section
//                     4.1 differ only in the score a candidate gets there.
//
// Logits are kept in the base-2 domain: s2 = sm_scale * log2(e) * (q . k), so
// weights are exp2(s2 - max2).
#pragma once

#include <cooperative_groups.h>

#include "tova_device.cuh"

namespace tova {

constexpr int TILE_ROWS = 16;       // cache rows per pipeline stage of the split kernel
constexpr int SPLIT_BUFFERS = 3;    // tile buffers of a split warp's ring (K and V tiles alternate)
constexpr int MAX_UNIT_HEADS = 8;   // query heads one split warp carries
constexpr int COMBINE_THREADS_TINY = 128;   // deferred victim/insert launches: small enough to slip in beside split warps
constexpr int COMBINE_THREADS_SMALL = 256;  // combine CTA size when many CTAs are in flight
constexpr int COMBINE_THREADS_LARGE = 512;  // ... when the batch is small: more loads in flight per sequence
constexpr int COMBINE_LOGIT_STAGE_BYTES = 96 * 1024;  // a combine CTA's [H][candidates] logits, staged if they fit
constexpr int COMBINE_ROW_STAGE_BYTES = 16 * 1024;  // new-token rows (k and v) staged in shared memory up to this size
constexpr int COMBINE_CLUSTER_MAX = 8;  // CTAs per sequence in the combine kernel (portable cluster size;
                                        // clusters of 16 were measured slower)
constexpr int MIN_CHUNK_ROWS = 32;      // smallest chunk the scratch is sized for
enum : int { COMBINE_ALL = 0, COMBINE_OUTPUTS = 1, COMBINE_EVICT = 2 };  // StepParams::mode

struct StepParams {
  // state
  void* K;            // [B,Hkv,cap,D]
  void* V;            // [B,Hkv,cap,D]
  int32_t* pos;       // [B,cap]
  int32_t* len;       // [B]
  // scratch
  float* logits;      // [B,H,ld]   base-2 logits of candidates 0..n (n = the new token)
  float2* part_ml;    // [B,H,pc]   (max2, sum) per chunk; entry n_chunks = the new token
  float* part_acc;    // [B,H,pc-1,D] un-normalised weighted V sums per chunk
  int32_t* status;    // [1]
  int32_t* cur_pos;   // [1] position of the token being processed (set by the split kernel)
  int32_t* last_slot; // [B] slot the previous step's token went to (-1: none), or null: no early prefetch
  float2* head_ml;    // [B,H] final (max2, sum) of every head, written with the outputs when fuse_out
  // this step
  const void* q;      // [B,H,D]
  const void* k_new;  // [B,Hkv,D]
  const void* v_new;  // [B,Hkv,D]
  float* out;         // [B,H,D]
  int32_t* evicted;   // [B] or null
  int32_t pos_t;      // the token's position, or < 0: previous token's position + 1
  // shape
  int32_t B, H, Hkv, G, cap, ld, pc;
  int32_t n;          // live rows before this step (same for every sequence)
  int32_t n_chunks;   // ceil(n / chunk_rows)
  int32_t chunk_rows; // rows per split warp, a multiple of TILE_ROWS
  int32_t hgroups;    // ceil(G / heads per split warp)
  int32_t nx;         // combine CTAs per sequence = cluster size (1..COMBINE_CLUSTER_MAX)
  int32_t cand_per_cta;  // candidates scored per combine CTA
  int32_t combine_threads;  // COMBINE_THREADS_TINY, _SMALL or _LARGE
  int32_t stage_logits;     // combine CTAs bulk-copy their block of logits to shared memory
  int32_t do_evict;   // n == cap and the policy is on
  int32_t fuse_out;   // the split kernel's warps of a (sequence, KV head, head group) form a cluster and write
                      // the outputs themselves; the combine kernel then only picks the victim
  int32_t policy;     // which row goes once the state is over capacity: POLICY_TOVA (lowest head-averaged weight,
                      // Algorithm 1) or POLICY_WINDOW (earliest position, Section 4.1)
  int32_t keep_first; // rows holding positions 0..keep_first-1 are never dropped ("+i" variants)
  int32_t merge_ctas; // fuse_out: CTAs (of up to 8 warps = chunks) per head group; > 1: they form a cluster (x)
  int32_t mode;       // combine kernel: 0 whole step, 1 outputs only, 2 victim + insert only
  void* k_stage;      // [B,Hkv,D] mode 1: copies of the new token's rows for a later mode-2 launch
  void* v_stage;
  float scale2;       // sm_scale * log2(e)
};

// ---------------------------------------------------------------------------
// output merge inside the split kernels (fuse_out)
// ---------------------------------------------------------------------------
// With at most SPLIT_MERGE_MAX_WARPS chunks, the split warps of one (sequence,
// KV head, head group) are launched as ONE CTA (blockDim = (32, n_chunks)):
// every warp still streams its own chunk through its own ring of buffers, then
// leaves its soft-max partial in shared memory where its tiles were; after one
// CTA barrier all threads merge the group's output quads - chunks in ascending
// order, then the new token (Eq. 7) - and write the final outputs and each
// head's (max2, sum).  No partial crosses global memory and no second kernel
// stands between the streaming and the caller's next kernel.
//
// Partial of a warp: per head D+4 floats: acc[D], max2, sum, -, -.  Warp 0
// also holds snew[g], the new token's logit per head.
constexpr int PART_STRIDE_EXTRA = 4;
constexpr int POLICY_TOVA = 0, POLICY_WINDOW = 1;
constexpr int SPLIT_MERGE_MAX_WARPS = 8;

template <int D>
__device__ __forceinline__ void empty_partial(float* part, int heads, int lane) {
  for (int i = lane; i < heads * (D + PART_STRIDE_EXTRA); i += 32)
    part[i] = (i % (D + PART_STRIDE_EXTRA) == D) ? -INFINITY : 0.f;
}

// Four consecutive elements of the new token's value row, as floats.
template <typename T>
__device__ __forceinline__ float4 load_quad(const T* src) {
  return make_float4((float)src[0], (float)src[1], (float)src[2], (float)src[3]);
}
template <>
__device__ __forceinline__ float4 load_quad<float>(const float* src) {
  return *reinterpret_cast<const float4*>(src);
}
template <>
__device__ __forceinline__ float4 load_quad<__nv_bfloat16>(const __nv_bfloat16* src) {
  const uint2 w = *reinterpret_cast<const uint2*>(src);   // 8-byte aligned: the quad starts at a multiple of 4 elements
  return make_float4(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u), __uint_as_float(w.y << 16),
                     __uint_as_float(w.y & 0xffff0000u));
}

// part0 / snew: warp 0's partial and new-token logits; warp w's partial lies
// warp_stride floats further per warp.  Called by every warp of the CTA.
template <typename T, int D>
__device__ __noinline__ void block_merge_outputs(float* out, float2* head_ml, const T* v_new_row, const float* part0,
                                                 int warp_stride, const float* snew, size_t bh0, int g_cnt) {
  constexpr int PS = D + PART_STRIDE_EXTRA;
  constexpr int NW = SPLIT_MERGE_MAX_WARPS;
  const int nw = (int)blockDim.y;
  const int tid = (int)(threadIdx.y * 32 + threadIdx.x);
  const int items = g_cnt * (D / 4);           // output quads of the group
  // the new token's value for this thread's first quad: on its way before the barrier
  float4 vq = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid < items) vq = load_quad<T>(v_new_row + (tid % (D / 4)) * 4);
  __syncthreads();                             // every warp's partial is in shared memory
  for (int it = tid; it < items; it += nw * 32) {
    const int g = it / (D / 4), d4 = it % (D / 4);
    if (it != tid) vq = load_quad<T>(v_new_row + d4 * 4);
    const float s_new = snew[g];
    float mr[NW], lr[NW];
    float M = s_new;
#pragma unroll
    for (int r = 0; r < NW; ++r) {
      if (r < nw) {
        mr[r] = part0[r * warp_stride + g * PS + D];
        lr[r] = part0[r * warp_stride + g * PS + D + 1];
        M = fmaxf(M, mr[r]);
      }
    }
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
#pragma unroll
    for (int r = 0; r < NW; ++r) {
      if (r < nw) {
        const float w = exp2_diff(mr[r], M);
        const float4 a = *reinterpret_cast<const float4*>(part0 + r * warp_stride + g * PS + d4 * 4);
        o.x = fmaf(a.x, w, o.x); o.y = fmaf(a.y, w, o.y); o.z = fmaf(a.z, w, o.z); o.w = fmaf(a.w, w, o.w);
        L = fmaf(lr[r], w, L);
      }
    }
    const float wn = exp2f(s_new - M);
    L += wn;
    const float iL = 1.f / L;
    o.x = fmaf(vq.x, wn, o.x) * iL; o.y = fmaf(vq.y, wn, o.y) * iL;
    o.z = fmaf(vq.z, wn, o.z) * iL; o.w = fmaf(vq.w, wn, o.w) * iL;
    reinterpret_cast<float4*>(out + (bh0 + g) * D)[d4] = o;
    if (d4 == 0) head_ml[bh0 + g] = make_float2(M, L);
  }
}

// The same across a thread-block cluster, for states of up to 8 x 8 chunks: the
// CTAs that share a head group (cluster dimension x, CTA r streams chunks 8r ..
// 8r+7) each merge their own warps' partials into one partial per head and
// SEND it to the CTA that owns that head (heads are dealt out over the CTAs of
// the cluster) - stores into the owner's shared memory (`cpart`, its inbox:
// [heads per CTA][CTAs][D+4] floats; CTA 0 adds the new token's logit) - then
// meet at ONE cluster barrier, after which every CTA merges what it received
// for its heads from its own shared memory and writes their outputs.  Nobody
// reads a peer's memory, so a CTA may leave as soon as it is done.  The inbox
// may only be written once its CTA runs: every thread arrives at the cluster
// barrier at kernel entry (split kernels) and waits for that phase here, just
// before the first remote store.
template <typename T, int D>
__device__ __noinline__ void cluster_merge_outputs(float* out, float2* head_ml, const T* v_new_row, const float* part0,
                                                   int warp_stride, float* snew0, float* cpart, size_t bh0,
                                                   int g_cnt) {
  namespace cg = cooperative_groups;
  cg::cluster_group cl = cg::this_cluster();
  constexpr int PS = D + PART_STRIDE_EXTRA;
  constexpr int NW = SPLIT_MERGE_MAX_WARPS;
  const int nw = (int)blockDim.y, nthreads = nw * 32;
  const int tid = (int)(threadIdx.y * 32 + threadIdx.x);
  const int ncta = (int)cl.num_blocks(), rank = (int)cl.block_rank();
  const int hpc = (g_cnt + ncta - 1) / ncta;   // heads per owning CTA
  const int items = g_cnt * (D / 4);           // output quads of the group
  // the new token's value for this thread's first quad of the second stage: on its way before the barriers
  const int my_items = min(hpc, max(g_cnt - rank * hpc, 0)) * (D / 4);
  float4 vq = make_float4(0.f, 0.f, 0.f, 0.f);
  if (tid < my_items) vq = load_quad<T>(v_new_row + (tid % (D / 4)) * 4);
  __syncthreads();                             // every warp's partial is in shared memory
  cluster_wait_acquire();                      // every CTA of the cluster has started: its inbox may be written
  float* inbox[COMBINE_CLUSTER_MAX];
#pragma unroll
  for (int r = 0; r < COMBINE_CLUSTER_MAX; ++r) inbox[r] = cl.map_shared_rank(cpart, r < ncta ? r : 0);
  for (int it = tid; it < items; it += nthreads) {
    const int g = it / (D / 4), d4 = it % (D / 4);
    float mr[NW], lr[NW];
    float M = -INFINITY;
#pragma unroll
    for (int r = 0; r < NW; ++r) {
      if (r < nw) {
        mr[r] = part0[r * warp_stride + g * PS + D];
        lr[r] = part0[r * warp_stride + g * PS + D + 1];
        M = fmaxf(M, mr[r]);
      }
    }
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
#pragma unroll
    for (int r = 0; r < NW; ++r) {
      if (r < nw) {
        const float w = exp2_diff(mr[r], M);
        const float4 a = *reinterpret_cast<const float4*>(part0 + r * warp_stride + g * PS + d4 * 4);
        o.x = fmaf(a.x, w, o.x); o.y = fmaf(a.y, w, o.y); o.z = fmaf(a.z, w, o.z); o.w = fmaf(a.w, w, o.w);
        L = fmaf(lr[r], w, L);
      }
    }
    const int owner = g / hpc, slot = g % hpc;
    float* dst = nullptr;
#pragma unroll
    for (int r = 0; r < COMBINE_CLUSTER_MAX; ++r)
      if (r == owner) dst = inbox[r];
    dst += (size_t)(slot * ncta + rank) * PS;
    *reinterpret_cast<float4*>(dst + d4 * 4) = o;
    if (d4 == 0) {
      dst[D] = M;
      dst[D + 1] = L;
      if (rank == 0) dst[D + 2] = snew0[g];    // the new token's logit travels with CTA 0's partial
    }
  }
  cluster_arrive_release();                    // orders the stores above before the barrier completes
  cluster_wait_acquire();
  for (int it = tid; it < my_items; it += nthreads) {
    const int slot = it / (D / 4), d4 = it % (D / 4);
    const int g = rank * hpc + slot;
    if (it != tid) vq = load_quad<T>(v_new_row + d4 * 4);
    const float* src = cpart + (size_t)slot * ncta * PS;
    const float s_new = src[D + 2];
    float mr[COMBINE_CLUSTER_MAX], lr[COMBINE_CLUSTER_MAX];
    float M = s_new;
#pragma unroll
    for (int r = 0; r < COMBINE_CLUSTER_MAX; ++r) {
      if (r < ncta) {
        mr[r] = src[r * PS + D];
        lr[r] = src[r * PS + D + 1];
        M = fmaxf(M, mr[r]);
      }
    }
    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
#pragma unroll
    for (int r = 0; r < COMBINE_CLUSTER_MAX; ++r) {
      if (r < ncta) {
        const float w = exp2_diff(mr[r], M);
        const float4 a = *reinterpret_cast<const float4*>(src + r * PS + d4 * 4);
        o.x = fmaf(a.x, w, o.x); o.y = fmaf(a.y, w, o.y); o.z = fmaf(a.z, w, o.z); o.w = fmaf(a.w, w, o.w);
        L = fmaf(lr[r], w, L);
      }
    }
    const float wn = exp2f(s_new - M);
    L += wn;
    const float iL = 1.f / L;
    o.x = fmaf(vq.x, wn, o.x) * iL; o.y = fmaf(vq.y, wn, o.y) * iL;
    o.z = fmaf(vq.z, wn, o.z) * iL; o.w = fmaf(vq.w, wn, o.w) * iL;
    reinterpret_cast<float4*>(out + (bh0 + g) * D)[d4] = o;
    if (d4 == 0) head_ml[bh0 + g] = make_float2(M, L);
  }
}

// One CTA per head group, or a cluster of them (merge_ctas > 1).
template <typename T, int D>
__device__ __forceinline__ void fused_merge(const StepParams& p, const T* v_new_row, const float* part0, int warp_stride,
                                            float* snew0, float* cpart, size_t bh0, int g_cnt) {
  if (p.merge_ctas > 1)
    cluster_merge_outputs<T, D>(p.out, p.head_ml, v_new_row, part0, warp_stride, snew0, cpart, bh0, g_cnt);
  else
    block_merge_outputs<T, D>(p.out, p.head_ml, v_new_row, part0, warp_stride, snew0, bh0, g_cnt);
}

// ---------------------------------------------------------------------------
// split kernel
// ---------------------------------------------------------------------------
// grid = (max(n_chunks,1), Hkv*hgroups, B), block = one warp.  The warp owns
// rows [c*chunk_rows, +chunk_rows) of one KV head and up to GU query heads of
// its group.  The operand tiles K_0 V_0 K_1 V_1 ... (16 rows each) travel through
// a ring of SPLIT_BUFFERS buffers: lane 0 issues the copy of operand tile u+NB
// into a buffer as soon as the warp has consumed tile u from it, so nothing but
// this warp ever waits on these barriers.
// Every lane reads 16 bytes of a row; LPR lanes cover a row, so the warp reads
// RPW = 32/LPR rows per pass and a tile takes NP = 16/RPW = LPR/2 passes.
template <typename T, int D, int GU, int GB, bool FUSED>
__global__ void __launch_bounds__(FUSED ? 32 * SPLIT_MERGE_MAX_WARPS : 32) tova_split_kernel(const StepParams p) {
  constexpr int EPL = Vec16<T>::N;          // elements per lane
  constexpr int RB = D * (int)sizeof(T);    // bytes per row
  constexpr int LPR = RB / 16;              // lanes per row
  constexpr int RPW = 32 / LPR;             // rows per pass
  constexpr int NP = TILE_ROWS / RPW;       // passes per tile (= LPR / 2)
  constexpr int TILE_BYTES = TILE_ROWS * RB;
  constexpr int NB = SPLIT_BUFFERS;
  static_assert(LPR >= 8 && LPR <= 32, "row must be 128..512 bytes");
  static_assert(GU % GB == 0, "head block must divide the unit");
  static_assert(NP * 2 == LPR, "a tile is half as many passes as lanes per row");

  // per warp: the ring and the weights of a tile, rounded up to 128 bytes
  constexpr int WARP_SMEM = (NB * TILE_BYTES + GU * TILE_ROWS * (int)sizeof(float) + 127) / 128 * 128;
  extern __shared__ __align__(128) unsigned char smem_all[];
  const int wib = FUSED ? threadIdx.y : 0;  // warp in block (FUSED: one CTA per head group, one warp per chunk)
  unsigned char* smem_raw = smem_all + (size_t)wib * WARP_SMEM;
  unsigned char* ring = smem_raw;                                    // [NB][TILE_BYTES]
  float* w_p = reinterpret_cast<float*>(smem_raw + NB * TILE_BYTES); // [GU][16] weights of a tile
  // fuse_out: once all tiles are consumed the ring holds this warp's partial [GU][D+4]
  // and (rank 0) the new token's logits [GU]
  float* part = reinterpret_cast<float*>(ring);
  static_assert((GU * (D + PART_STRIDE_EXTRA) + GU) * sizeof(float) <= (size_t)NB * TILE_BYTES, "partial fits the ring");
  __shared__ __align__(8) uint64_t bars_all[SPLIT_MERGE_MAX_WARPS][NB];
  uint64_t* bars = bars_all[wib];
  const float* part0 = reinterpret_cast<const float*>(smem_all);    // warp 0's partial
  __shared__ float snew_s[MAX_UNIT_HEADS];                          // the new token's logit per head (chunk 0's warp)
  // merge_ctas > 1: this CTA's inbox for the cluster merge, behind the rings
  float* cpart = reinterpret_cast<float*>(smem_all + (size_t)(FUSED ? blockDim.y : 1) * WARP_SMEM);

  // Merge across a cluster: peers will store into this CTA's shared memory; report in (see cluster_merge_outputs).
  if (FUSED && p.merge_ctas > 1) cluster_arrive_release();

  const int lane = threadIdx.x;
  const int lig = lane % LPR;   // lane in row group
  const int sub = lane / LPR;   // which of the RPW rows of a pass
  const int c = FUSED ? (int)(blockIdx.x * blockDim.y) + wib : (int)blockIdx.x, b = blockIdx.z;
  const int kvh = blockIdx.y / p.hgroups, hg = blockIdx.y % p.hgroups;
  const int g_begin = hg * GU;
  const int g_cnt = min(GU, p.G - g_begin);                 // real heads of this unit
  const int row_begin = c * p.chunk_rows;
  const int rows = min(max(p.n - row_begin, 0), p.chunk_rows);
  const int ntiles = (rows + TILE_ROWS - 1) / TILE_ROWS;
  // After the transposing reduction lanes lig and lig^NP both hold the logit of
  // tile row (lig % NP) * RPW + sub; the lower one of the pair "owns" it.
  const int my_row = (lig % NP) * RPW + sub;
  const bool owner = lig < NP;

  if (lane == 0) {
#pragma unroll
    for (int s = 0; s < NB; ++s) mbar_init(&bars[s], 1);
    mbar_fence_init();
  }
  __syncwarp();

  const unsigned char* k_src =
      static_cast<const unsigned char*>(p.K) + (((size_t)b * p.Hkv + kvh) * p.cap + row_begin) * RB;
  const unsigned char* v_src =
      static_cast<const unsigned char*>(p.V) + (((size_t)b * p.Hkv + kvh) * p.cap + row_begin) * RB;

  const int n_ops = 2 * ntiles;        // operand tiles: u = 2t is K_t, u = 2t+1 is V_t
  const uint64_t stream_policy = l2_policy_evict_first();
  auto issue = [&](int u) {            // lane 0 only
    const int t = u >> 1;
    const uint32_t bytes = (uint32_t)min(TILE_ROWS, rows - t * TILE_ROWS) * RB;
    uint64_t* bar = &bars[u % NB];
    mbar_expect_tx(bar, bytes);
    bulk_g2s_hint(ring + (size_t)(u % NB) * TILE_BYTES, ((u & 1) ? v_src : k_src) + (size_t)t * TILE_BYTES, bytes,
                  bar, stream_policy);
  };
  // Early prefetch.  The previous step's combine kernel may still be running:
  // the only thing it writes to the state is one row per sequence (the slot its
  // token went to, recorded in last_slot).  Every other row is final, so the
  // first tiles can be fetched now, before the dependency wait; if the one row
  // in question lies in them, it is fetched again after the wait (patch below).
  const bool early = p.last_slot != nullptr;
  if (early && lane == 0) {
    for (int u = 0; u < min(NB, n_ops); ++u) issue(u);
  }

  // Nothing above reads global memory through this thread; below we read what
  // earlier kernels in the stream wrote.
  pdl_wait();
  pdl_launch_dependents();

  if (c == 0 && blockIdx.y == 0 && blockIdx.z == 0 && lane == 0)
    *p.cur_pos = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;
  if (!early && lane == 0) {
    for (int u = 0; u < min(NB, n_ops); ++u) issue(u);
  }
  // Every global load of the prologue is issued before the first one is used:
  // the row that may have changed, q of the unit's heads (kept packed, 16 bytes
  // per head and lane) and, for chunk 0's warp, the new token's key.
  const T* qbase = static_cast<const T*>(p.q) + ((size_t)b * p.H + (size_t)kvh * p.G + g_begin) * D;
  const size_t bh0 = (size_t)b * p.H + (size_t)kvh * p.G + g_begin;
  const int ls = early ? __ldcg(p.last_slot + b) : -1;
  uint4 qpk[GU];
#pragma unroll
  for (int g = 0; g < GU; ++g)
    qpk[g] = *reinterpret_cast<const uint4*>(qbase + (size_t)min(g, g_cnt - 1) * D + lig * EPL);
  uint4 knw = make_uint4(0u, 0u, 0u, 0u);
  if (c == 0)
    knw = *reinterpret_cast<const uint4*>(static_cast<const T*>(p.k_new) + ((size_t)b * p.Hkv + kvh) * D + lig * EPL);

  int patch_row = -1;              // row of this chunk that must be fetched again, if any
  if (ls >= row_begin && ls < row_begin + rows) patch_row = ls - row_begin;
  // Re-fetches row patch_row of operand tile u (already landed) from global memory.
  auto patch = [&](int u, unsigned char* tile, const unsigned char* src) {
    const int t = u >> 1;
    if (patch_row >= 0 && u < NB && patch_row / TILE_ROWS == t) {
      if (lane < LPR)
        *reinterpret_cast<uint4*>(tile + (size_t)(patch_row % TILE_ROWS) * RB + lane * 16) =
            __ldcg(reinterpret_cast<const uint4*>(src + (size_t)patch_row * RB) + lane);
      __syncwarp();
    }
  };

  // The new token (candidate n): its logit per head, by the warp of chunk 0
  // while its first copies are in flight.
  if (c == 0) {
    float kf[EPL];
    Vec16<T>::unpack(knw, kf);
#pragma unroll
    for (int g = 0; g < GU; ++g) {
      if (g < g_cnt) {
        float qf[EPL];
        Vec16<T>::unpack(qpk[g], qf);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
        for (int o = LPR / 2; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        s *= p.scale2;
        if (lane == 0) {
          p.logits[(bh0 + g) * p.ld + p.n] = s;
          if (FUSED) snew_s[g] = s;
          else p.part_ml[(bh0 + g) * p.pc + p.n_chunks] = make_float2(s, 1.f);
        }
      }
    }
    if (FUSED && p.k_stage && hg == 0 && lane < LPR) {  // copies for a deferred eviction (the caller may reuse k and v)
      const size_t w16 = ((size_t)b * p.Hkv + kvh) * LPR + lane;
      static_cast<uint4*>(p.k_stage)[w16] = static_cast<const uint4*>(p.k_new)[w16];
      static_cast<uint4*>(p.v_stage)[w16] = static_cast<const uint4*>(p.v_new)[w16];
    }
  }
  if (ntiles == 0) {          // empty state: only the new token exists
    if (FUSED) {
      empty_partial<D>(part, GU, lane);
      fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
    }
    return;
  }


  float m[GU], l[GU], acc[GU][EPL];
#pragma unroll
  for (int g = 0; g < GU; ++g) {
    m[g] = -INFINITY;
    l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) acc[g][e] = 0.f;
  }

  bool failed = false;
  int t = 0;
  for (; t < ntiles; ++t) {
    const int uk = 2 * t, uv = 2 * t + 1;
    const int nvalid = min(TILE_ROWS, rows - t * TILE_ROWS);
    unsigned char* kt = ring + (size_t)(uk % NB) * TILE_BYTES;
    unsigned char* vt = ring + (size_t)(uv % NB) * TILE_BYTES;

    // ---- logits of the tile's rows, GB heads at a time -------------------------
    if (!warp_wait(&bars[uk % NB], (uint32_t)(uk / NB) & 1u)) { failed = true; break; }
    patch(uk, kt, k_src);
    float s[GU];
#pragma unroll
    for (int g0 = 0; g0 < GU; g0 += GB) {
      float qf[GB][EPL];
#pragma unroll
      for (int gb = 0; gb < GB; ++gb) Vec16<T>::unpack(qpk[g0 + gb], qf[gb]);
      float part[GB][NP];
#pragma unroll
      for (int i = 0; i < NP; ++i) {
        const int r = i * RPW + sub;
        float kf[EPL];
        Vec16<T>::unpack(*reinterpret_cast<const uint4*>(kt + (size_t)r * RB + lig * 16), kf);
#pragma unroll
        for (int gb = 0; gb < GB; ++gb) {
          float a = 0.f;
#pragma unroll
          for (int e = 0; e < EPL; ++e) a = fmaf(qf[gb][e], kf[e], a);
          part[gb][i] = a;
        }
      }
#pragma unroll
      for (int gb = 0; gb < GB; ++gb) {
        float v = transpose_reduce<NP>(part[gb], lig % NP);
        v = (v + __shfl_xor_sync(0xffffffffu, v, NP)) * p.scale2;
        // rows past the live range hold stale shared memory: mask them out
        s[g0 + gb] = (my_row < nvalid) ? v : -INFINITY;
      }
    }
    // the K buffer is free: refill it with the tile after next
    __syncwarp();
    if (lane == 0 && uk + NB < n_ops) {
      fence_proxy_async_smem();
      issue(uk + NB);
    }

    // ---- online soft-max update, weights of the tile to shared memory --------
#pragma unroll
    for (int g = 0; g < GU; ++g) {
      if (g < g_cnt && owner && my_row < nvalid)
        p.logits[(bh0 + g) * p.ld + row_begin + t * TILE_ROWS + my_row] = s[g];
      const float m_new = fmaxf(m[g], warp_max(s[g]));
      const float corr = exp2_diff(m[g], m_new);
      const float e = exp2_diff(s[g], m_new);
      // l stays a per-lane partial sum (rows this lane owns); it is folded once at the end
      l[g] = fmaf(l[g], corr, owner ? e : 0.f);
      m[g] = m_new;
      if (corr != 1.f) {             // warp-uniform (the max is a warp reduction): rare after the first tiles
#pragma unroll
        for (int k = 0; k < EPL; ++k) acc[g][k] *= corr;
      }
      if (owner) w_p[g * TILE_ROWS + my_row] = e;
    }
    __syncwarp();

    // ---- weighted V sum --------------------------------------------------------
    if (!warp_wait(&bars[uv % NB], (uint32_t)(uv / NB) & 1u)) { failed = true; break; }
    patch(uv, vt, v_src);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      const int r = i * RPW + sub;
      if (r < nvalid) {
        float vf[EPL];
        Vec16<T>::unpack(*reinterpret_cast<const uint4*>(vt + (size_t)r * RB + lig * 16), vf);
#pragma unroll
        for (int g = 0; g < GU; ++g) {
          const float w = w_p[g * TILE_ROWS + r];
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[g][e] = fmaf(w, vf[e], acc[g][e]);
        }
      }
    }
    __syncwarp();
    if (lane == 0 && uv + NB < n_ops) {
      fence_proxy_async_smem();
      issue(uv + NB);
    }
  }

  if (failed) {
    // Give copies still in flight a last bounded chance to land before the
    // shared memory is released, and report.
    for (int u = 2 * t; u < min(2 * t + NB, n_ops); ++u) warp_wait(&bars[u % NB], (uint32_t)(u / NB) & 1u);
    if (lane == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    if (FUSED) {           // the other warps wait at the CTA barrier: join them with an empty partial
      empty_partial<D>(part, GU, lane);
      fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
    }
    return;
  }

  __syncwarp();                 // fuse_out: the partial goes where the tiles were
  // ---- fold the RPW row groups of the warp, write the chunk partial -----------
#pragma unroll
  for (int g = 0; g < GU; ++g) {
#pragma unroll
    for (int e = 0; e < EPL; ++e)
#pragma unroll
      for (int o = LPR; o < 32; o <<= 1) acc[g][e] += __shfl_xor_sync(0xffffffffu, acc[g][e], o);
    l[g] = warp_sum(l[g]);
    if (g < g_cnt && sub == 0) {
      float* dst = FUSED ? part + g * (D + PART_STRIDE_EXTRA) + lig * EPL
                              : p.part_acc + ((bh0 + g) * (size_t)(p.pc - 1) + c) * D + lig * EPL;
#pragma unroll
      for (int e = 0; e < EPL; e += 4)
        *reinterpret_cast<float4*>(dst + e) = make_float4(acc[g][e], acc[g][e + 1], acc[g][e + 2], acc[g][e + 3]);
      if (lane == 0) {
        if (FUSED) {
          part[g * (D + PART_STRIDE_EXTRA) + D] = m[g];
          part[g * (D + PART_STRIDE_EXTRA) + D + 1] = l[g];
        } else {
          p.part_ml[(bh0 + g) * p.pc + c] = make_float2(m[g], l[g]);
        }
      }
    }
  }
  if (FUSED) fused_merge<T, D>(p, static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + kvh) * D, part0, WARP_SMEM / 4, snew_s,
                        cpart, bh0, g_cnt);
}


// ---------------------------------------------------------------------------
// combine-and-evict kernel
// ---------------------------------------------------------------------------
// grid = (nx, B) with the nx CTAs of a sequence forming one thread-block cluster
// (nx <= 8), block = CT threads.  The step lasts microseconds, so the
// kernel is built around dependent memory round trips, not throughput: every
// global load a thread will need (chunk partials, logits of its candidates,
// weighted V sums of its output element, the candidate's position, the words of
// the new token's row) is issued up front into registers, in one round trip.
//   1. each CTA rebuilds every head's global (max2, 1/sum) from the partials;
//   2. CTA x writes its 1/nx share of the H*D attention outputs (Eq. 7);
//   3. CTA x scores candidates [x*cand_per_cta, +cand_per_cta): the mean over
//      heads of the soft-max weights (Algorithm 1), in a fixed order, and sends
//      its lowest (value, index, position) to CTA 0's shared memory;
//   4. after one cluster barrier CTA 0 takes the overall arg-min - lowest index
//      on ties - and replaces that row by the new token in K, V and the position
//      table (Eq. 9, in place).  No global atomics, no CTA waits on a flag.
// smem: float2 pml[H][np]; float hM[H], hInvL[H], hLc[H], sc[CT]; then, in
// CTA 0 only, the new token's k and v rows of all KV heads (bulk-copied in at
// the start when they fit COMBINE_ROW_STAGE_BYTES); then the CTA's
// [H][cand_per_cta] block of logits (bulk-copied in at the start when the host
// says it fits).
// 64 registers per thread: CTAs of the next kernel can share the SM with them.
// MODE (COMBINE_ALL / COMBINE_OUTPUTS / COMBINE_EVICT) is a template parameter:
// with warm data the kernel stalls mostly on instruction fetch, so every launch
// should carry only the code it runs.
template <typename T, int D, int CT, int MODE>
__global__ void __launch_bounds__(CT, 1024 / CT) tova_combine_kernel(const StepParams p) {
  namespace cg = cooperative_groups;
  constexpr bool BIG = false;
  constexpr int ML = BIG ? 4 : 2;    // partial pairs prefetched per thread
  constexpr int LG = BIG ? 16 : 8;   // logits prefetched per thread
  constexpr int AC = BIG ? 8 : 2;    // weighted V sums (float4) prefetched per thread
  extern __shared__ __align__(16) float csm[];
  const int np = p.n_chunks + 1;   // partials per head: the chunks, then the new token
  float2* pml = reinterpret_cast<float2*>(csm);                  // [H][np]
  float* hM = csm + 2 * (size_t)p.H * np;                        // [H]
  float* hInvL = hM + p.H;                                       // [H]
  float* hLc = hInvL + p.H;                                      // [H] -max2 - log2(sum * H)
  float* sc = hLc + p.H;                                         // [CT]
  unsigned char* row_stage = reinterpret_cast<unsigned char*>(
      (reinterpret_cast<uintptr_t>(sc + CT) + 15) & ~uintptr_t(15));     // [2][Hkv*D*sizeof(T)]
  __shared__ __align__(8) uint64_t row_bar;
  __shared__ __align__(8) uint64_t lg_bar;
  __shared__ float red_v[CT / 32];
  __shared__ int red_i[CT / 32];
  __shared__ int red_p[CT / 32];
  __shared__ float4 best_of[COMBINE_CLUSTER_MAX];  // CTA 0's copy collects every CTA's minimum
  __shared__ int s_victim;

  const int x = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  // geometry (no memory access)
  // (all the divisors below are powers of two: shifts and masks, no integer division)
  int lg_wp = 0;                   // wp = candidates per pass, a power of two <= CT
  while ((1 << lg_wp) < p.cand_per_cta && (1 << lg_wp) < CT) ++lg_wp;
  const int wp = 1 << lg_wp;
  const int hs_n = CT >> lg_wp;    // threads sharing one candidate's heads
  const int jl = tid & (wp - 1), hs = tid >> lg_wp;
  const int j_begin = x * p.cand_per_cta;
  const int j_end = min(j_begin + p.cand_per_cta, p.n + 1);
  // When a victim is due, CTA 0 is on the critical path (arg-min, insert): if
  // the output merge is light (few chunks), the output elements are shared among
  // its peers and written after they arrive at the cluster barrier.
  const bool score = p.do_evict && MODE != COMBINE_OUTPUTS;          // this launch picks a victim
  const bool late_out = score && MODE == COMBINE_ALL && p.nx > 1 && p.n_chunks <= 8;   // only when the merge is light
  const int out_ctas = late_out ? p.nx - 1 : p.nx;
  const int out_x = late_out ? x - 1 : x;      // -1: no share
  // Output work item = (head, 4 consecutive dims, slice of the chunks): S lanes
  // next to each other share an output quad, each merging every S-th chunk with
  // 16-byte loads; their sums are folded by shuffles.
  const int items4 = p.H * (D / 4);
  const int out_threads = out_ctas * CT;
  int lg_S = 0;
  while ((2 << lg_S) <= 32 && (2 << lg_S) * items4 <= out_threads && (2 << lg_S) <= p.n_chunks) ++lg_S;
  const int S = 1 << lg_S;
  const int work = items4 * S;                 // a multiple of 32 whenever S > 1
  const bool fused = p.fuse_out != 0;          // outputs and per-head (max, sum) already came from the split kernel
  const int g0 = (out_x < 0 || MODE == COMBINE_EVICT || fused) ? work : out_x * CT + tid;
  constexpr int RB16 = D * (int)sizeof(T) / 16;  // 16-byte words per row
  const int row_words = p.Hkv * RB16;
  int lg_np = 0;                   // partials per head rounded up to a power of two: thread i -> (i >> lg_np, i & mask)
  while ((1 << lg_np) < np) ++lg_np;
  const int total_ml = p.H << lg_np;
  const uint32_t row_bytes = (uint32_t)row_words * 16u;          // all KV heads of one operand
  const bool staged = (x == 0) && MODE != COMBINE_OUTPUTS && 2 * row_bytes <= (uint32_t)COMBINE_ROW_STAGE_BYTES;
  // staged logits: rows of cand_per_cta floats (a multiple of 4), one per head
  float* lg_stage = reinterpret_cast<float*>(
      row_stage + (2 * row_bytes <= (uint32_t)COMBINE_ROW_STAGE_BYTES ? 2 * row_bytes : 0));
  const int lg_cols = max(min(p.cand_per_cta, p.ld - j_begin), 0);   // floats per head row actually copied
  const bool lg_staged = score && p.stage_logits && lg_cols > 0;
  if (tid == 0) {
    mbar_init(&row_bar, 1);
    mbar_init(&lg_bar, 1);
    mbar_fence_init();
  }
  __syncthreads();
  // The block minima travel to CTA 0 through distributed shared memory, which
  // may only be touched once its CTA runs: the CTAs of a cluster are resident
  // together but need not start together.  Everybody reports in here (without
  // waiting) and checks that all have done so just before that store.
  if (score) cluster_arrive_release();

  pdl_wait();
  pdl_launch_dependents();
  if (staged && tid == 0) {        // the new token's rows, on their way while everything else happens
    mbar_expect_tx(&row_bar, 2 * row_bytes);
    bulk_g2s(row_stage, static_cast<const unsigned char*>(p.k_new) + (size_t)b * row_bytes, row_bytes, &row_bar);
    bulk_g2s(row_stage + row_bytes, static_cast<const unsigned char*>(p.v_new) + (size_t)b * row_bytes, row_bytes,
             &row_bar);
  }
  if (lg_staged && warp == 1) {    // this CTA's block of logits: one bulk copy per head
    if (lane == 0) mbar_expect_tx(&lg_bar, (uint32_t)p.H * (uint32_t)lg_cols * 4u);
    __syncwarp();
    for (int h = lane; h < p.H; h += 32)
      bulk_g2s(lg_stage + (size_t)h * p.cand_per_cta, p.logits + ((size_t)b * p.H + h) * p.ld + j_begin,
               (uint32_t)lg_cols * 4u, &lg_bar);
  }

  // ---- 0. every load this thread needs, issued back to back ---------------------
  const int pos_t = *p.cur_pos;
  float2 r_ml[ML];
#pragma unroll
  for (int u = 0; u < ML; ++u) {
    const int i = tid + u * CT;
    const int h = i >> lg_np, cc = i & ((1 << lg_np) - 1);
    r_ml[u] = (!fused && i < total_ml && cc < np) ? p.part_ml[((size_t)b * p.H + h) * p.pc + cc]
                                                  : make_float2(0.f, 0.f);
  }
  float r_lg[LG];
  int r_pos = pos_t;               // position held by this thread's first candidate
  {
    const int j = j_begin + jl;
    const bool live = score && j < j_end;
    const float* lg = p.logits + (size_t)b * p.H * p.ld + j;
#pragma unroll
    for (int u = 0; u < LG; ++u) {
      const int h = hs + u * hs_n;
      r_lg[u] = (live && !lg_staged && h < p.H) ? lg[(size_t)h * p.ld] : 0.f;
    }
    if (live && hs == 0 && j < p.cap) r_pos = p.pos[(size_t)b * p.cap + j];
  }
  float4 r_acc[AC];
  if (MODE != COMBINE_EVICT && g0 < work) {
    const int it = g0 >> lg_S, cs = g0 & (S - 1);
    const int h = it / (D / 4), d4 = it % (D / 4);
    const float4* acc = reinterpret_cast<const float4*>(p.part_acc + ((size_t)b * p.H + h) * (size_t)(p.pc - 1) * D) + d4;
#pragma unroll
    for (int u = 0; u < AC; ++u) {
      const int i = cs + u * S;
      r_acc[u] = (i < p.n_chunks) ? acc[(size_t)i * (D / 4)] : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  } else {
#pragma unroll
    for (int u = 0; u < AC; ++u) r_acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
  }

  // Writes the new token's k and v into row `slot` of every KV head (CTA 0 only).
  auto insert_row = [&](int slot) {
    bool from_smem = staged;
    if (staged && !mbar_wait_bounded(&row_bar, 0)) {
      from_smem = false;           // fall back to reading the rows again
      if (tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    }
    const uint4* ks = from_smem ? reinterpret_cast<const uint4*>(row_stage)
                                : static_cast<const uint4*>(p.k_new) + (size_t)b * row_words;
    const uint4* vs = from_smem ? reinterpret_cast<const uint4*>(row_stage + row_bytes)
                                : static_cast<const uint4*>(p.v_new) + (size_t)b * row_words;
    for (int i = tid; i < row_words; i += CT) {
      const size_t dst = (((size_t)b * p.Hkv + i / RB16) * p.cap + slot) * RB16 + i % RB16;
      static_cast<uint4*>(p.K)[dst] = ks[i];
      static_cast<uint4*>(p.V)[dst] = vs[i];
    }
  };

  // ---- 1. global max and sum of every head ---------------------------------------------
  if (fused) {
    for (int h = tid; h < p.H; h += CT) {
      const float2 e = p.head_ml[(size_t)b * p.H + h];
      hM[h] = e.x;
      hInvL[h] = __frcp_rn(e.y);
      hLc[h] = -e.x - __log2f(e.y * (float)p.H);
    }
    __syncthreads();
  } else {
#pragma unroll
    for (int u = 0; u < ML; ++u) {
      const int i = tid + u * CT;
      const int h = i >> lg_np, cc = i & ((1 << lg_np) - 1);
      if (i < total_ml && cc < np) pml[h * np + cc] = r_ml[u];
    }
    for (int i = tid + ML * CT; i < total_ml; i += CT) {
      const int h = i >> lg_np, cc = i & ((1 << lg_np) - 1);
      if (cc < np) pml[h * np + cc] = p.part_ml[((size_t)b * p.H + h) * p.pc + cc];
    }
    __syncthreads();
    {
      // a group of lph lanes per head, at most 8 partials per lane
      int lg_lph = 0;
      while ((1 << lg_lph) < 32 && (8 << lg_lph) < np) ++lg_lph;
      const int lph = 1 << lg_lph;
      const int hpp = CT >> lg_lph;                  // heads per pass
      const int sub_l = tid & (lph - 1);
      for (int h0 = 0; h0 < p.H; h0 += hpp) {        // uniform trip count: the shuffles need whole warps
        const int h = h0 + (tid >> lg_lph);
        const bool hv = h < p.H;
        const float2* ml = pml + (size_t)(hv ? h : 0) * np;
        float M = -INFINITY, L = 0.f;
        for (int i = sub_l; i < np; i += lph) M = fmaxf(M, ml[i].x);
        for (int o = lph >> 1; o >= 1; o >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, o));
        for (int i = sub_l; i < np; i += lph) L = fmaf(ml[i].y, exp2f(ml[i].x - M), L);   // M is finite: the new token's partial is
        for (int o = lph >> 1; o >= 1; o >>= 1) L += __shfl_xor_sync(0xffffffffu, L, o);
        if (hv && sub_l == 0) {
          hM[h] = M;
          hInvL[h] = __frcp_rn(L);
          hLc[h] = -M - __log2f(L * (float)p.H);
        }
      }
    }
    __syncthreads();
  }

  // ---- 2. this CTA's share of the attention output --------------------------------
  auto write_outputs = [&]() {
    for (int g = g0; g < work; g += out_threads) {   // whole warps run the same trips (see `work`)
      const int it = g >> lg_S, cs = g & (S - 1);
      const int h = it / (D / 4), d4 = it % (D / 4);
      const size_t bh = (size_t)b * p.H + h;
      const float2* ml = pml + (size_t)h * np;
      const float4* acc = reinterpret_cast<const float4*>(p.part_acc + bh * (size_t)(p.pc - 1) * D) + d4;
      const float M = hM[h];
      float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
      int i = cs;
      if (g == g0) {
#pragma unroll
        for (int u = 0; u < AC; ++u) {
          if (i < p.n_chunks) {
            const float w = exp2f(ml[i].x - M);
            o.x = fmaf(r_acc[u].x, w, o.x); o.y = fmaf(r_acc[u].y, w, o.y);
            o.z = fmaf(r_acc[u].z, w, o.z); o.w = fmaf(r_acc[u].w, w, o.w);
          }
          i += S;
        }
      }
#pragma unroll 4
      for (; i < p.n_chunks; i += S) {
        const float4 a = acc[(size_t)i * (D / 4)];
        const float w = exp2f(ml[i].x - M);
        o.x = fmaf(a.x, w, o.x); o.y = fmaf(a.y, w, o.y); o.z = fmaf(a.z, w, o.z); o.w = fmaf(a.w, w, o.w);
      }
      for (int off = S >> 1; off >= 1; off >>= 1) {
        o.x += __shfl_xor_sync(0xffffffffu, o.x, off); o.y += __shfl_xor_sync(0xffffffffu, o.y, off);
        o.z += __shfl_xor_sync(0xffffffffu, o.z, off); o.w += __shfl_xor_sync(0xffffffffu, o.w, off);
      }
      if (cs == 0) {
        const T* vn = static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + h / p.G) * D + d4 * 4;
        const float w = exp2f(ml[p.n_chunks].x - M), iL = hInvL[h];
        o.x = fmaf((float)vn[0], w, o.x) * iL; o.y = fmaf((float)vn[1], w, o.y) * iL;
        o.z = fmaf((float)vn[2], w, o.z) * iL; o.w = fmaf((float)vn[3], w, o.w) * iL;
        reinterpret_cast<float4*>(p.out + bh * D)[d4] = o;
      }
    }
  };
  if (MODE != COMBINE_EVICT && !late_out) write_outputs();

  if (MODE == COMBINE_OUTPUTS) {
    // The victim is chosen by a later launch, possibly after the caller has
    // reused its k/v buffers: keep copies of the new token's rows.
    if (x == 0) {
      for (int i = tid; i < row_words; i += CT) {
        static_cast<uint4*>(p.k_stage)[(size_t)b * row_words + i] =
            static_cast<const uint4*>(p.k_new)[(size_t)b * row_words + i];
        static_cast<uint4*>(p.v_stage)[(size_t)b * row_words + i] =
            static_cast<const uint4*>(p.v_new)[(size_t)b * row_words + i];
      }
    }
    return;
  }

  if (!p.do_evict) {
    // g(t) = min(t, k) not yet reached: the new token takes the next free row.
    if (x == 0) {
      insert_row(p.n);
      if (tid == 0) {
        p.pos[(size_t)b * p.cap + p.n] = pos_t;
        p.len[b] = p.n + 1;
        if (p.last_slot) p.last_slot[b] = p.n;
        if (p.evicted) p.evicted[b] = -1;
      }
    }
    return;
  }

  // ---- 3. head-averaged weight of this CTA's candidates ---------------------------
  // thread = (candidate jl of a pass, head slice hs); passes of wp candidates
  float val = INFINITY;
  int idx = 0x7fffffff;
  int cpos = pos_t;                // position held by the best candidate (the new token holds pos_t)
  bool lg_ok = true;
  if (lg_staged && !mbar_wait_bounded(&lg_bar, 0)) {
    lg_ok = false;                 // read the logits from global memory instead
    if (tid == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
  }
  for (int j0 = j_begin; j0 < j_end; j0 += wp) {
    const int j = j0 + jl;
    const bool live = j < j_end;
    float a = 0.f;
    if (live) {
      const float* lg = p.logits + (size_t)b * p.H * p.ld + j;
      if (lg_staged && lg_ok) {
        const float* sl = lg_stage + (j - j_begin);
#pragma unroll 8
        for (int h = hs; h < p.H; h += hs_n) a += exp2f(sl[(size_t)h * p.cand_per_cta] + hLc[h]);
      } else if (j0 == j_begin && !lg_staged) {
#pragma unroll
        for (int u = 0; u < LG; ++u) {
          const int h = hs + u * hs_n;
          if (h < p.H) a += exp2f(r_lg[u] + hLc[h]);
        }
#pragma unroll 4
        for (int h = hs + LG * hs_n; h < p.H; h += hs_n) a += exp2f(lg[(size_t)h * p.ld] + hLc[h]);
      } else {
#pragma unroll 4
        for (int h = hs; h < p.H; h += hs_n) a += exp2f(lg[(size_t)h * p.ld] + hLc[h]);
      }
    }
    if (hs_n > 1) {                // uniform over the CTA
      sc[tid] = a;
      __syncthreads();
      if (hs == 0) {
        a = 0.f;
        for (int k = 0; k < hs_n; ++k) a += sc[k * wp + jl];
      }
      __syncthreads();
    }
    if (hs == 0 && live) {
      float v = a;                   // the 1/H of the mean is folded into hLc
      int pj = 0;
      const bool by_pos = p.policy != POLICY_TOVA || p.keep_first > 0;   // uniform
      if (by_pos) {                  // the other policies look at the position the candidate holds
        pj = (j0 == j_begin) ? r_pos : ((j < p.cap) ? p.pos[(size_t)b * p.cap + j] : pos_t);
        // Window: the earliest position goes.  Ages of droppable rows are below the capacity
        // (the policy is fixed while the state is empty), so the float is exact.
        if (p.policy == POLICY_WINDOW) v = (float)(pj - pos_t);
        if (pj < p.keep_first) v = INFINITY;     // one of the first i token states: never dropped
      }
      if (v < val) {               // passes go up in j: strict < keeps the lowest index
        val = v;
        idx = j;
        cpos = by_pos ? pj : ((j0 == j_begin) ? r_pos : ((j < p.cap) ? p.pos[(size_t)b * p.cap + j] : pos_t));
      }
    }
  }
  // lowest (value, index) of the block
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    const int op = __shfl_xor_sync(0xffffffffu, cpos, o);
    if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; cpos = op; }
  }
  if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; red_p[warp] = cpos; }
  __syncthreads();
  cg::cluster_group cluster = cg::this_cluster();
  cluster_wait_acquire();          // every CTA of the cluster has started (arrival at kernel entry)
  if (tid == 0) {
    for (int w = 1; w < CT / 32; ++w)
      if (red_v[w] < val || (red_v[w] == val && red_i[w] < idx)) { val = red_v[w]; idx = red_i[w]; cpos = red_p[w]; }
    // into CTA 0's shared memory (distributed shared memory store)
    *cluster.map_shared_rank(&best_of[x], 0) = make_float4(val, __int_as_float(idx), __int_as_float(cpos), 0.f);
  }

  // ---- 4. one cluster barrier; CTA 0 takes the arg-min, evicts, inserts -----------
  __syncwarp();
  cluster_arrive_release();        // orders the store above before the barrier completes
  if (x != 0) {                    // peers: nobody reads their shared memory; their outputs are off the critical path
    if (MODE == COMBINE_ALL && late_out) write_outputs();
    return;
  }
  cluster_wait_acquire();
  if (warp == 0) {
    float bv = INFINITY;
    int bi = 0x7fffffff, bp = pos_t;
    if (lane < p.nx) {
      const float4 e = best_of[lane];
      bv = e.x; bi = __float_as_int(e.y); bp = __float_as_int(e.z);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      const int op = __shfl_xor_sync(0xffffffffu, bp, o);
      if (ov < bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; bp = op; }
    }
    if (lane == 0) {
      if (bi < 0 || bi > p.cap) { atomicExch(p.status, DEV_ERR_BAD_VICTIM); bi = p.cap; bp = pos_t; }
      s_victim = bi;
      if (bi < p.cap) p.pos[(size_t)b * p.cap + bi] = pos_t;
      if (p.last_slot) p.last_slot[b] = (bi < p.cap) ? bi : -1;
      if (p.evicted) p.evicted[b] = bp;  // the new token's own position if it dropped itself
    }
  }
  __syncthreads();
  const int victim = s_victim;
  if (victim < p.cap) insert_row(victim);
  else if (staged) mbar_wait_bounded(&row_bar, 0);  // the staged copy must land before the CTA leaves
}

// Host-buffer steps: q, k and v are fetched from page-locked host memory once,
// with coalesced 16-byte reads, into device staging (the split kernel's warps
// would each read q over the bus otherwise).
__global__ void tova_fetch_inputs_kernel(uint4* dq, const uint4* hq, int nq, uint4* dk, const uint4* hk, uint4* dv,
                                         const uint4* hv, int nk) {
  const int stride = gridDim.x * blockDim.x;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < nq + 2 * nk; i += stride) {
    if (i < nq) dq[i] = hq[i];
    else if (i < nq + nk) dk[i - nq] = hk[i - nq];
    else dv[i - nq - nk] = hv[i - nq - nk];
  }
}

// Empty state at init: length 0, positions -1, status 0.
__global__ void tova_init_kernel(int32_t* pos, int32_t* len, int32_t* last_slot, int32_t* status,
                                 int32_t* cur_pos, int B, int cap) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < (size_t)B * cap) pos[i] = -1;
  if (i < (size_t)B) { len[i] = 0; last_slot[i] = -1; }
  if (i == 0) { *status = 0; *cur_pos = -1; }
}

}  // namespace tova
