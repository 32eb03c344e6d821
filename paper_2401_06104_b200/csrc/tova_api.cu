// Host side of the C ABI declared in include/tova.h: argument checks, the
// layout of the caller-provided device block, launch configuration.  Every
// step of the decode path runs in the kernels of tova_kernels.cuh and
// tova_split_mma.cuh, the bulk fill of a prompt in those of tova_fill.cuh;
// there is no CPU fallback.
#include "../../include/tova.h"

#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <type_traits>

#include "tova_kernels.cuh"
#include "tova_split_mma.cuh"
#include "tova_fill.cuh"
#include "tova_fill_tc.cuh"
#include "tova_units.cuh"
#include "tova_chunk.cuh"
#include "tova_shard.cuh"
#include "tova_poscomp.cuh"

namespace {

constexpr size_t ALIGN = 256;
inline size_t align_up(size_t x) { return (x + ALIGN - 1) / ALIGN * ALIGN; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct Layout {
  size_t K, V, pos, len, last_slot, logits, part_ml, part_acc, head_ml, status, cur_pos;
  size_t st_q, st_k, st_v, st_out, st_ev;  // staging for host-buffer calls
  size_t df_k, df_v;                       // the new token's rows kept for a deferred eviction
  size_t upos, uacc;                       // per-KV-head slot tables and accumulated scores (head-wise policies, H2O)
  size_t upart, uticket;                   // slice minima and ticket counters of the unit-policy kernel
  size_t shard_words;                      // epoch and ticket of the sharded step
  size_t total;
  int ld, pc;
};

bool config_ok(const tova_config* c, int* why) {
  if (!c) { *why = TOVA_ERR_NULL; return false; }
  if (c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->capacity < 1 ||
      c->n_q_heads % c->n_kv_heads != 0 || c->batch > 65535 || c->n_kv_heads > 65535 ||
      c->n_q_heads > 4096 || c->capacity > (1 << 24)) {
    *why = TOVA_ERR_BAD_SHAPE;
    return false;
  }
  if ((c->head_dim != 64 && c->head_dim != 128) ||
      (c->dtype != TOVA_DTYPE_FP32 && c->dtype != TOVA_DTYPE_BF16)) {
    *why = TOVA_ERR_UNSUPPORTED;
    return false;
  }
  if (!(c->sm_scale >= 0.f) || !std::isfinite(c->sm_scale)) { *why = TOVA_ERR_BAD_SHAPE; return false; }
  return true;
}

Layout make_layout(const tova_config& c) {
  Layout L{};
  const size_t B = c.batch, H = c.n_q_heads, Hkv = c.n_kv_heads, D = c.head_dim, cap = c.capacity;
  const size_t E = c.dtype == TOVA_DTYPE_BF16 ? 2 : 4;
  L.ld = (int)((cap + 1 + 3) / 4 * 4);
  // scratch is sized for the smallest chunk (32 rows per split warp)
  L.pc = (int)((cap + tova::MIN_CHUNK_ROWS - 1) / tova::MIN_CHUNK_ROWS) + 1;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.K = take(B * Hkv * cap * D * E);
  L.V = take(B * Hkv * cap * D * E);
  L.pos = take(B * cap * 4);
  L.len = take(B * 4);
  L.last_slot = take(B * 4);
  L.logits = take(B * H * L.ld * 4);
  L.part_ml = take(B * H * L.pc * 8);
  L.part_acc = take(B * H * (size_t)(L.pc - 1) * D * 4);
  L.head_ml = take(B * H * 8);
  L.status = take(4);
  L.cur_pos = take(4);
  L.st_q = take(B * H * D * E);
  L.st_k = take(B * Hkv * D * E);
  L.st_v = take(B * Hkv * D * E);
  L.st_out = take(B * H * D * 4);
  L.st_ev = take(B * Hkv * 4);
  L.df_k = take(B * Hkv * D * E);
  L.df_v = take(B * Hkv * D * E);
  L.upos = take(B * Hkv * cap * 4);
  L.uacc = take(B * Hkv * cap * 4);
  L.upart = take(B * Hkv * tova::UNIT_MAX_SLICES * sizeof(tova::UnitPartial));
  L.uticket = take(B * Hkv * 4);
  L.shard_words = take(8);
  L.total = off;
  return L;
}

// Caller-provided scratch of the chunked prompt path (tova_cache_set_prefill_workspace).
struct ChunkLayout {
  size_t Kst, Vst, lg, rt, ml, death, slot_token, first, total;
  int ldc;
};

ChunkLayout make_chunk_layout(const tova_config& c) {
  ChunkLayout L{};
  const size_t B = c.batch, H = c.n_q_heads, Hkv = c.n_kv_heads, D = c.head_dim, cap = c.capacity;
  const size_t CT = tova::CHUNK_TOKENS;
  L.ldc = (int)((cap + 3) / 4 * 4 + CT);      // state columns, then (16-byte aligned) the chunk's own
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.Kst = take(B * Hkv * CT * D * 2);
  L.Vst = take(B * Hkv * CT * D * 2);
  L.lg = take(B * H * CT * L.ldc * 4);
  L.rt = take(B * H * CT * 8);
  L.ml = take(B * H * CT * 8);
  L.death = take(B * L.ldc * 4);
  L.slot_token = take(B * cap * 4);
  L.first = take(4);
  L.total = off;
  return L;
}

}  // namespace

struct tova_cache {
  tova_config cfg;
  CUtensorMap map_k, map_v;  // tiled views of K and V for the tensor-core split kernel
  bool use_mma;
  CUtensorMap fill_map_k, fill_map_v;  // the same matrices in boxes of 64 rows, for the bulk fill of a prompt
  bool fill_maps;
  int bulk_fill;   // 0: prompts token by token; 1: bulk fill, tcgen05 kernel where head_dim is 128; 2: bulk fill, warp-level MMA kernel
  int policy, keep_first;  // which row is dropped once the state is over capacity (tova_cache_set_policy)
  int units;               // 0: the layer policies of the combine kernel; else units that own rows (1 or Hkv)
  int recent;              // H2O: size of the window of most recent tokens that always stay
  bool fuse_merge;      // the split warps of a head group form one CTA and merge the outputs themselves
  // deferred eviction: victim choice and insert run on a side stream, overlapping later work
  bool deferred, pending;
  cudaStream_t side;
  cudaEvent_t ev_fork, ev_join;
  Layout lay;
  unsigned char* base;
  // chunked prompt path: caller-provided workspace and tiled views of its staging tiles
  // position compression: caller-provided workspace (table of cosines and sines, rotated query, positions)
  unsigned char* poscomp_ws;
  tova::PosCompParams poscomp;
  // state sharded by KV head over several ranks (tova_cache_set_shard)
  bool shard_on, shard_scored;
  tova::ShardParams shard;
  unsigned char* chunk_ws;
  int chunk_cluster;       // 0: automatic; 1, 2, 4, 8: CTAs per sequence of the deletion kernel; -1: the one-CTA kernel
  int chunk_two_barriers;  // 1: the cluster kernel with two barriers per token even where the one-barrier kernel fits
  ChunkLayout chunk_lay;
  CUtensorMap chunk_map_k, chunk_map_v;
  int32_t len;          // rows per sequence (host mirror; sequences move in lock step)
  int64_t launches;
  int chunk_rows;       // rows of the state per split warp
  int sm_count;
  int device;
  float scale2;
  size_t elem, row_bytes;
};

namespace {

using tova::StepParams;

// The tensor-core split kernel serves bf16 states whose query group is a real
// contraction (G >= 4 rows of the 16-row MMA tile); everything else - MHA above
// all, which does one flop per byte - runs on the plain ALUs.
inline bool wants_mma(const tova_config& cfg) {
  return cfg.dtype == TOVA_DTYPE_BF16 && cfg.n_q_heads / cfg.n_kv_heads >= 4;
}

// Heads one split warp carries (GU) and heads per pass over a tile (GB).
inline int unit_heads_alu(int G) { return G <= 1 ? 1 : G == 2 ? 2 : G <= 4 ? 4 : tova::MAX_UNIT_HEADS; }
inline int unit_heads(const tova_config& cfg) {
  return wants_mma(cfg) ? tova::MMA_UNIT_HEADS : unit_heads_alu(cfg.n_q_heads / cfg.n_kv_heads);
}

inline size_t split_smem_bytes(const tova_config& cfg) {
  const size_t rb = (size_t)cfg.head_dim * (cfg.dtype == TOVA_DTYPE_BF16 ? 2 : 4);
  if (wants_mma(cfg)) return (size_t)tova::SPLIT_BUFFERS * tova::TILE_ROWS * rb + 1024;
  const int gu = unit_heads(cfg);
  return ((size_t)tova::SPLIT_BUFFERS * tova::TILE_ROWS * rb + sizeof(float) * gu * tova::TILE_ROWS + 127) / 128 * 128;
}

// Merge inside the split kernel: the warps of a head group's chunks form one CTA
// of up to 8 warps, or merge_ctas such CTAs in a cluster along x.
inline void split_launch_shape(const StepParams& p, dim3& grid, dim3& block) {
  block = dim3(32);
  if (p.fuse_out) {
    block.y = (grid.x + p.merge_ctas - 1) / p.merge_ctas;
    grid.x = p.merge_ctas;
  }
}
// Launch attributes of a split kernel: programmatic dependent launch, plus the cluster when CTAs merge across.
inline int split_launch_attrs(const StepParams& p, cudaLaunchAttribute* at) {
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  if (!p.fuse_out || p.merge_ctas <= 1) return 1;
  at[1].id = cudaLaunchAttributeClusterDimension;
  at[1].val.clusterDim.x = p.merge_ctas;
  at[1].val.clusterDim.y = 1;
  at[1].val.clusterDim.z = 1;
  return 2;
}
// Shared memory behind the rings for a CTA's inbox of the cluster merge: one partial from every CTA of the
// cluster for each of the heads this CTA owns (heads dealt out over the CTAs, rounded up).
inline size_t cluster_inbox_bytes(int heads, int D) {
  return sizeof(float) * (size_t)(heads + tova::COMBINE_CLUSTER_MAX) * (D + tova::PART_STRIDE_EXTRA);
}
inline size_t cluster_partial_bytes(const StepParams& p, int heads, int D) {
  return (p.fuse_out && p.merge_ctas > 1) ? cluster_inbox_bytes(heads, D) : 0;
}

template <typename T, int D, int GU, int GB, bool FUSED>
cudaError_t launch_split_f(int dev, const StepParams& p, dim3 grid, cudaStream_t st) {
  const size_t rb = (size_t)D * sizeof(T);
  const size_t warp_smem =
      ((size_t)tova::SPLIT_BUFFERS * tova::TILE_ROWS * rb + sizeof(float) * GU * tova::TILE_ROWS + 127) / 128 * 128;
  dim3 block;
  split_launch_shape(p, grid, block);
  const size_t smem = warp_smem * block.y + cluster_partial_bytes(p, GU, D);
  auto kern = tova::tova_split_kernel<T, D, GU, GB, FUSED>;
  static std::atomic<bool> attr_set[64];  // per instantiation and device: the attribute is per function
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(
        kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
        (int)(warp_smem * tova::SPLIT_MERGE_MAX_WARPS + cluster_inbox_bytes(GU, D)));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  cfg.attrs = at;
  cfg.numAttrs = split_launch_attrs(p, at);
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <typename T, int D, int GU, int GB>
cudaError_t launch_split(int dev, const StepParams& p, dim3 grid, cudaStream_t st) {
  return p.fuse_out ? launch_split_f<T, D, GU, GB, true>(dev, p, grid, st)
                    : launch_split_f<T, D, GU, GB, false>(dev, p, grid, st);
}

template <typename T, int D>
cudaError_t launch_split_g(int dev, int G, const StepParams& p, dim3 grid, cudaStream_t st) {
  constexpr bool wide = (D * sizeof(T) == 512);  // fp32, D = 128: 32 partial sums per head and lane
  switch (unit_heads_alu(G)) {
    case 1: return launch_split<T, D, 1, 1>(dev, p, grid, st);
    case 2: return launch_split<T, D, 2, wide ? 1 : 2>(dev, p, grid, st);
    case 4: return launch_split<T, D, 4, wide ? 1 : 4>(dev, p, grid, st);
    default: return launch_split<T, D, 8, wide ? 1 : 2>(dev, p, grid, st);
  }
}

// Dynamic shared memory of the combine kernel: all (max, sum) partials of a
// sequence, per-head max and 1/sum, one float per thread, and the new token's
// rows when they are small enough to be staged.
inline size_t combine_smem_bytes(int H, int n_partials, int threads, size_t row_bytes, size_t logit_bytes) {
  size_t b = sizeof(float) * (2 * (size_t)H * n_partials + 3 * (size_t)H + threads) + 16;
  if (2 * row_bytes <= (size_t)tova::COMBINE_ROW_STAGE_BYTES) b += 2 * row_bytes;
  return b + logit_bytes;
}
constexpr size_t COMBINE_SMEM_LIMIT = 200 * 1024;   // opt-in maximum of the combine kernel
constexpr size_t COMBINE_BASE_LIMIT = 100 * 1024;   // partials + rows; staged logits come on top
// upper bound used when choosing chunk sizes (largest CTA, rows staged)
inline size_t combine_smem_bound(int H, int n_partials) {
  return combine_smem_bytes(H, n_partials, tova::COMBINE_THREADS_LARGE, 0, 0) + tova::COMBINE_ROW_STAGE_BYTES;
}

template <typename T, int D, int CT, int MODE>
cudaError_t launch_combine_ct(int dev, const StepParams& p, cudaStream_t st, bool use_pdl) {
  const size_t row_bytes = (size_t)p.Hkv * D * sizeof(T);
  const size_t logit_bytes = p.stage_logits ? (size_t)p.H * p.cand_per_cta * sizeof(float) : 0;
  const size_t smem = combine_smem_bytes(p.H, p.n_chunks + 1, CT, row_bytes, logit_bytes);
  auto kern = tova::tova_combine_kernel<T, D, CT, MODE>;
  static std::atomic<bool> attr_set[64];
  if (!attr_set[dev & 63]) {
    cudaError_t e =
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)COMBINE_SMEM_LIMIT);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(p.nx, p.B);
  cfg.blockDim = dim3(CT);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (use_pdl) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    ++na;
  }
  if (MODE != tova::COMBINE_OUTPUTS) {  // the CTAs of one sequence form a cluster (needed to pick the victim)
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = p.nx;
    at[na].val.clusterDim.y = 1;
    at[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, kern, p);
}

template <typename T, int D>
cudaError_t launch_combine(int dev, const StepParams& p, cudaStream_t st, bool use_pdl = true) {
  constexpr int CL = tova::COMBINE_THREADS_LARGE, CS = tova::COMBINE_THREADS_SMALL, CY = tova::COMBINE_THREADS_TINY;
  const bool large = p.combine_threads == CL;
  switch (p.mode) {
    case tova::COMBINE_OUTPUTS:
      return large ? launch_combine_ct<T, D, CL, tova::COMBINE_OUTPUTS>(dev, p, st, use_pdl)
                   : launch_combine_ct<T, D, CS, tova::COMBINE_OUTPUTS>(dev, p, st, use_pdl);
    case tova::COMBINE_EVICT:
      if (p.combine_threads == CY) return launch_combine_ct<T, D, CY, tova::COMBINE_EVICT>(dev, p, st, use_pdl);
      return large ? launch_combine_ct<T, D, CL, tova::COMBINE_EVICT>(dev, p, st, use_pdl)
                   : launch_combine_ct<T, D, CS, tova::COMBINE_EVICT>(dev, p, st, use_pdl);
    default:
      return large ? launch_combine_ct<T, D, CL, tova::COMBINE_ALL>(dev, p, st, use_pdl)
                   : launch_combine_ct<T, D, CS, tova::COMBINE_ALL>(dev, p, st, use_pdl);
  }
}

template <int D, bool TWO, bool FUSED>
cudaError_t launch_split_mma_t(int dev, const StepParams& p, const CUtensorMap& mk, const CUtensorMap& mv, dim3 grid,
                               cudaStream_t st) {
  const size_t warp_smem = (size_t)tova::SPLIT_BUFFERS * tova::TILE_ROWS * D * 2;
  dim3 block;
  split_launch_shape(p, grid, block);
  const size_t smem = warp_smem * block.y + 1024 + cluster_partial_bytes(p, tova::MMA_UNIT_HEADS, D);
  auto kern = tova::tova_split_mma_kernel<D, TWO, FUSED>;
  static std::atomic<bool> attr_set[64];
  if (!attr_set[dev & 63]) {
    cudaError_t e = cudaFuncSetAttribute(
        kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
        (int)(warp_smem * tova::SPLIT_MERGE_MAX_WARPS + 1024 + cluster_inbox_bytes(tova::MMA_UNIT_HEADS, D)));
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, 100);
    if (e != cudaSuccess) return e;
    attr_set[dev & 63] = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  cfg.attrs = at;
  cfg.numAttrs = split_launch_attrs(p, at);
  return cudaLaunchKernelEx(&cfg, kern, p, mk, mv);
}

template <int D>
cudaError_t launch_split_mma(int dev, const StepParams& p, const CUtensorMap& mk, const CUtensorMap& mv, dim3 grid,
                             cudaStream_t st) {
  if (p.fuse_out)
    return p.G > 8 ? launch_split_mma_t<D, true, true>(dev, p, mk, mv, grid, st)
                   : launch_split_mma_t<D, false, true>(dev, p, mk, mv, grid, st);
  return p.G > 8 ? launch_split_mma_t<D, true, false>(dev, p, mk, mv, grid, st)
                 : launch_split_mma_t<D, false, false>(dev, p, mk, mv, grid, st);
}

void set_combine_threads(StepParams& p, int ct);
constexpr size_t POSCOMP_SMEM_LIMIT = 200 * 1024;

template <typename T, int D>
cudaError_t launch_step(tova_cache* c, const StepParams& p, cudaStream_t st, bool defer) {
  dim3 grid(p.n_chunks > 0 ? p.n_chunks : 1, p.Hkv * p.hgroups, p.B);
  cudaError_t e;
  if (c->pending) {  // the previous token's deferred insert must land before the state is read
    e = cudaStreamWaitEvent(st, c->ev_join, 0);
    if (e != cudaSuccess) return e;
    c->pending = false;
  }
  if (c->poscomp_ws) {
    // Position compression: new positions and their cosines/sines per sequence, the rotating streaming kernel,
    // then the ordinary combine kernel (merge, outputs, victim, insert of the un-rotated key).
    static std::atomic<bool> pc_configured[64];
    if (c->device >= 0 && c->device < 64 && !pc_configured[c->device]) {
      if ((e = cudaFuncSetAttribute(tova::tova_poscomp_kernel<T, D>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)POSCOMP_SMEM_LIMIT)) != cudaSuccess) return e;
      pc_configured[c->device] = true;
    }
    // (the table's sines and cosines in double are the bulk of that kernel: a sequence's entries are shared out
    //  among as many blocks as one wave of the GPU holds, at least 8 table rows each)
    int pc_blocks = std::max(1, c->sm_count / p.B);
    pc_blocks = std::max(1, std::min(pc_blocks, (p.n + 1 + 7) / 8));
    tova::tova_poscomp_kernel<T, D><<<dim3(p.B, pc_blocks), tova::POSCOMP_THREADS, tova::poscomp_smem_bytes(p.cap, D), st>>>(
        p, c->poscomp);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    switch (tova::rope_unit_heads(p.G)) {
      case 1: tova::tova_split_rope_kernel<T, D, 1><<<grid, 32, 0, st>>>(p, c->poscomp); break;
      case 2: tova::tova_split_rope_kernel<T, D, 2><<<grid, 32, 0, st>>>(p, c->poscomp); break;
      default: tova::tova_split_rope_kernel<T, D, 4><<<grid, 32, 0, st>>>(p, c->poscomp); break;
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if ((e = launch_combine<T, D>(c->device, p, st)) != cudaSuccess) return e;
    c->launches += 3;
    return cudaSuccess;
  }
  if constexpr (std::is_same<T, __nv_bfloat16>::value) {
    e = c->use_mma ? launch_split_mma<D>(c->device, p, c->map_k, c->map_v, grid, st)
                   : launch_split_g<T, D>(c->device, p.G, p, grid, st);
  } else {
    e = launch_split_g<T, D>(c->device, p.G, p, grid, st);
  }
  if (e != cudaSuccess) return e;
  if (c->shard_on) {
    // This rank's heads of a sharded layer: outputs as on one GPU, then (once a row is due to go) the rank's partial
    // head sums into every rank's table.  Victim and insert follow in tova_decode_step_commit.
    int n_launch = 1;
    if (!p.fuse_out) {
      StepParams pa = p;
      pa.mode = tova::COMBINE_OUTPUTS;
      pa.k_stage = c->base + c->lay.df_k;
      pa.v_stage = c->base + c->lay.df_v;
      pa.stage_logits = 0;
      if ((e = launch_combine<T, D>(c->device, pa, st)) != cudaSuccess) return e;
      ++n_launch;
    }
    if (p.do_evict) {
      tova::tova_shard_scores_kernel<<<dim3(p.nx, p.B), tova::SHARD_THREADS, sizeof(float) * p.H, st>>>(p, c->shard);
      if ((e = cudaGetLastError()) != cudaSuccess) return e;
      ++n_launch;
    }
    c->launches += n_launch;
    return cudaSuccess;
  }
  if (c->units > 0) {
    // Policies whose rows are owned per unit (a KV head, or the layer with accumulated scores): outputs as for
    // the layer policy, then one thread block per (unit, sequence) scores, picks and inserts.
    int n_launch = 2;
    if (!p.fuse_out) {
      StepParams pa = p;
      pa.mode = tova::COMBINE_OUTPUTS;
      pa.k_stage = c->base + c->lay.df_k;
      pa.v_stage = c->base + c->lay.df_v;
      pa.stage_logits = 0;
      if ((e = launch_combine<T, D>(c->device, pa, st)) != cudaSuccess) return e;
      n_launch = 3;
    }
    tova::UnitParams up{};
    up.units = c->units;
    up.table = reinterpret_cast<int32_t*>(c->base + (c->units == 1 ? c->lay.pos : c->lay.upos));
    up.acc = reinterpret_cast<float*>(c->base + c->lay.uacc);
    up.recent = c->recent;
    up.h2o = (c->policy == tova::POLICY_H2O_LAYER || c->policy == tova::POLICY_H2O_HEAD) ? 1 : 0;
    up.part = reinterpret_cast<tova::UnitPartial*>(c->base + c->lay.upart);
    up.ticket = reinterpret_cast<int32_t*>(c->base + c->lay.uticket);
    const int nh = c->units == 1 ? p.H : p.G;
    // Few (unit, sequence) pairs: cut each pair's candidates into slices of at least 256, up to two blocks per SM.
    int slices = (2 * c->sm_count) / (c->units * p.B);
    slices = std::min(slices, (p.n + 1 + 255) / 256);
    slices = std::max(1, std::min(slices, tova::UNIT_MAX_SLICES));
    // Deferred: victim choice and insert run on the side stream, from the copies of the new token's rows that the
    // streaming kernel (or the outputs launch) left in the cache block, and overlap whatever the caller enqueues next.
    StepParams pu = p;
    cudaStream_t ust = st;
    if (defer) {
      if ((e = cudaEventRecord(c->ev_fork, st)) != cudaSuccess) return e;
      if ((e = cudaStreamWaitEvent(c->side, c->ev_fork, 0)) != cudaSuccess) return e;
      pu.k_new = c->base + c->lay.df_k;
      pu.v_new = c->base + c->lay.df_v;
      ust = c->side;
    }
    tova::tova_unit_policy_kernel<T, D><<<dim3(c->units, p.B, slices), tova::UNIT_THREADS, sizeof(float) * nh, ust>>>(pu, up);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    if (defer) {
      if ((e = cudaEventRecord(c->ev_join, c->side)) != cudaSuccess) return e;
      c->pending = true;
    }
    c->launches += n_launch;
    return cudaSuccess;
  }
  if (p.fuse_out) {
    // The split kernel has written the outputs; what is left is the victim and
    // the insert, on the caller's stream or (deferred) on the side stream.
    StepParams pb = p;
    pb.mode = tova::COMBINE_EVICT;
    if (!defer) {
      e = launch_combine<T, D>(c->device, pb, st);
      if (e != cudaSuccess) return e;
      c->launches += 2;
      return cudaSuccess;
    }
    if ((e = cudaEventRecord(c->ev_fork, st)) != cudaSuccess) return e;
    if ((e = cudaStreamWaitEvent(c->side, c->ev_fork, 0)) != cudaSuccess) return e;
    pb.k_new = p.k_stage;
    pb.v_new = p.v_stage;
    pb.k_stage = pb.v_stage = nullptr;
    // Off the critical path, but every CTA of this launch that sits on an SM keeps one of the next split
    // kernel's 8-warp CTAs from becoming resident there: as few CTAs as about 32 logits per thread allow
    // (measured at mistral k=256, B=32: 256 -> 96 CTAs, 11.2 -> 10.5 us per step).
    {
      const long long score_loads = (long long)(p.n + 1) * p.H;
      int nx = (int)((score_loads + 32LL * tova::COMBINE_THREADS_TINY - 1) / (32LL * tova::COMBINE_THREADS_TINY));
      if (nx < 1) nx = 1;
      if (nx < p.nx && p.do_evict) {
        pb.nx = nx;
        pb.cand_per_cta = ((p.n + 1 + nx - 1) / nx + 3) / 4 * 4;
      }
    }
    set_combine_threads(pb, (long long)pb.H * pb.cand_per_cta / tova::COMBINE_THREADS_TINY <= 40
                                ? tova::COMBINE_THREADS_TINY : tova::COMBINE_THREADS_SMALL);
    e = launch_combine<T, D>(c->device, pb, c->side, /*use_pdl=*/false);
    if (e != cudaSuccess) return e;
    if ((e = cudaEventRecord(c->ev_join, c->side)) != cudaSuccess) return e;
    c->pending = true;
    c->launches += 2;
    return cudaSuccess;
  }
  if (!defer) {
    e = launch_combine<T, D>(c->device, p, st);
    if (e != cudaSuccess) return e;
    c->launches += 2;
    return cudaSuccess;
  }
  // Deferred eviction: the outputs (what the caller's next kernels need) come
  // from a launch on the caller's stream; victim choice and insert follow on the
  // side stream and overlap whatever the caller enqueues next.
  StepParams pa = p;
  pa.mode = tova::COMBINE_OUTPUTS;
  pa.k_stage = c->base + c->lay.df_k;
  pa.v_stage = c->base + c->lay.df_v;
  // Outputs-only launch: half-size CTAs once the batch would otherwise fill the
  // register files and keep the next split kernel from becoming resident early.
  if ((long long)p.B * p.nx > c->sm_count) set_combine_threads(pa, tova::COMBINE_THREADS_SMALL);
  pa.stage_logits = 0;
  e = launch_combine<T, D>(c->device, pa, st);
  if (e != cudaSuccess) return e;
  if ((e = cudaEventRecord(c->ev_fork, st)) != cudaSuccess) return e;
  if ((e = cudaStreamWaitEvent(c->side, c->ev_fork, 0)) != cudaSuccess) return e;
  StepParams pb = p;
  pb.mode = tova::COMBINE_EVICT;
  pb.k_new = pa.k_stage;
  pb.v_new = pa.v_stage;
  // Victim + insert launch: off the critical path, so small CTAs that fit beside
  // the next layer's split warps (128 threads unless that means long serial scoring).
  set_combine_threads(pb, (long long)p.H * p.cand_per_cta / tova::COMBINE_THREADS_TINY <= 40
                              ? tova::COMBINE_THREADS_TINY : tova::COMBINE_THREADS_SMALL);
  e = launch_combine<T, D>(c->device, pb, c->side, /*use_pdl=*/false);
  if (e != cudaSuccess) return e;
  if ((e = cudaEventRecord(c->ev_join, c->side)) != cudaSuccess) return e;
  c->pending = true;
  c->launches += 3;
  return cudaSuccess;
}

// Rows of the state per split warp.  Every SM holds `per_sm` split warps at a
// time (shared memory and registers).  Measured on B200 over the model-shaped
// workloads: 128-row chunks are best whenever they give at least ~0.8 warps per
// slot (several rounds of short warps beat one round of long ones: the tail
// is shorter and the load spreads better); with fewer, 64-row chunks double
// the warps; 32-row chunks lose more in the combine kernel (twice the
// partials) than they gain.  Larger chunks only where the combine kernel's
// shared memory would not hold all partials of a sequence.
bool fused_merge_fits(const tova_config& cfg, int chunk_rows, int sm_count);

int pick_chunk_rows(const tova_config& cfg, int sm_count) {
  const size_t smem = split_smem_bytes(cfg) + 1024 /* per-CTA reserve */ + 64;
  long long per_sm = (long long)(227 * 1024) / (long long)smem;
  // registers bound the resident warps too (figures from ptxas for these kernels)
  const int G0 = cfg.n_q_heads / cfg.n_kv_heads;
  const long long by_regs = wants_mma(cfg) ? (G0 > 8 ? 12 : 21) : (G0 <= 1 ? 25 : G0 == 2 ? 16 : G0 <= 4 ? 12 : 8);
  if (per_sm > by_regs) per_sm = by_regs;
  if (per_sm > 32) per_sm = 32;
  if (per_sm < 1) per_sm = 1;
  const long long slots = per_sm * sm_count;
  const long long hgroups = (G0 + unit_heads(cfg) - 1) / unit_heads(cfg);
  const long long pairs = (long long)cfg.batch * cfg.n_kv_heads * hgroups;
  auto units = [&](int cr) { return pairs * ((cfg.capacity + (long long)cr - 1) / cr); };
  int cr = 128;
  if (10 * units(128) < 8 * slots) cr = 64;
  if (cr == 64 && cfg.capacity <= 256 && 10 * units(64) < 8 * slots) cr = 32;  // short states: partials are few anyway
  // Tensor-core kernel with at least 1.5 head groups per SM: one CTA of 8 warps per group fills the GPU by
  // itself, so the state is cut into exactly 8 chunks however long (measured at mistral B=32: k=4096 96.1 ->
  // 90.2 us, k=2048 even; with fewer groups, or on the ALU kernel, shorter chunks in more CTAs win).
  if (wants_mma(cfg) && 2 * pairs >= 3LL * sm_count) {
    const int cr8 = (int)(((cfg.capacity + 7) / 8 + 31) / 32 * 32);
    if (cr8 > cr) cr = cr8;
  }
  // More than 8 x 8 chunks cannot merge inside the streaming kernel.  Where chunks long enough to get back under
  // that limit keep the launch within what clusters merge well (fused_merge_fits), take them: at 4 sequences x 4 KV
  // heads x 8192 rows the step is 18.0 us with 128-row chunks in clusters against 35.5 us with 64-row chunks and
  // partials through global memory (16384 rows: 32.1 against 47.7 us).
  {
    const int limit = tova::SPLIT_MERGE_MAX_WARPS * tova::COMBINE_CLUSTER_MAX;
    int cr2 = cr;
    while (cr2 < 8192 && (cfg.capacity + cr2 - 1) / cr2 > limit) cr2 *= 2;
    if (cr2 != cr && (cfg.capacity + cr2 - 1) / cr2 <= limit && fused_merge_fits(cfg, cr2, sm_count)) cr = cr2;
  }
  while (cr <= 8192 && combine_smem_bound(cfg.n_q_heads, (int)((cfg.capacity + cr - 1) / cr) + 1) > COMBINE_BASE_LIMIT)
    cr *= 2;
  return cr <= 8192 ? cr : -1;  // -1: no chunk size keeps the combine kernel's shared memory within its limit
}

// Whether the split kernel merges the chunk partials itself: always when one CTA
// of 8 warps covers the state; with up to 8 such CTAs per head group (a
// cluster) only while the launch is a few waves of CTAs at most - beyond that
// single-warp CTAs, which the hardware hands out one by one, stream better.
bool fused_merge_fits(const tova_config& cfg, int chunk_rows, int sm_count) {
  const int chunks = (cfg.capacity + chunk_rows - 1) / chunk_rows;
  if (chunks <= tova::SPLIT_MERGE_MAX_WARPS) return true;
  if (chunks > tova::SPLIT_MERGE_MAX_WARPS * tova::COMBINE_CLUSTER_MAX) return false;
  const int G = cfg.n_q_heads / cfg.n_kv_heads;
  const long long hgroups = (G + unit_heads(cfg) - 1) / unit_heads(cfg);
  const long long ctas = (long long)cfg.batch * cfg.n_kv_heads * hgroups *
                         ((chunks + tova::SPLIT_MERGE_MAX_WARPS - 1) / tova::SPLIT_MERGE_MAX_WARPS);
  // measured: the tensor-core kernel keeps gaining from the in-kernel merge up to several waves of CTAs
  // (mistral k=2048/4096 at batch 32: -7 % / -2 % per step), the ALU kernel only within one resident wave
  return ctas <= (wants_mma(cfg) ? 8LL : 2LL) * sm_count;
}

// CTA size of a combine launch, and with it whether a CTA's logits are staged
// through shared memory (bulk copies): only when a thread would otherwise need
// several dependent batches of loads for them.
void set_combine_threads(StepParams& p, int ct) {
  p.combine_threads = ct;
  const long long per_thread = (long long)p.H * p.cand_per_cta / ct;
  p.stage_logits = p.do_evict && per_thread > 3 * 8 &&
                   (size_t)p.H * p.cand_per_cta * sizeof(float) <= (size_t)tova::COMBINE_LOGIT_STAGE_BYTES;
}

// Launch geometry of one step for n live rows.
void fill_geometry(StepParams& p, const tova_config& cfg, int n, int chunk_rows, int sm_count) {
  p.B = cfg.batch; p.H = cfg.n_q_heads; p.Hkv = cfg.n_kv_heads; p.G = cfg.n_q_heads / cfg.n_kv_heads;
  p.cap = cfg.capacity;
  p.n = n;
  p.chunk_rows = chunk_rows;
  p.n_chunks = (n + chunk_rows - 1) / chunk_rows;
  p.hgroups = (p.G + unit_heads(cfg) - 1) / unit_heads(cfg);
  p.do_evict = (n == cfg.capacity) ? 1 : 0;
  // Combine CTAs per sequence (one cluster): 512-thread CTAs (two per SM)
  // while they all fit on the GPU at once, else 256-thread CTAs (four per SM).
  // Per thread: about one output quad and at most 8 logits per pass.
  const int cl_max = tova::COMBINE_CLUSTER_MAX;
  const long long ctas = (long long)cfg.batch * cl_max;
  const int ct = ctas <= 2LL * sm_count ? tova::COMBINE_THREADS_LARGE : tova::COMBINE_THREADS_SMALL;
  const int lg = 8;
  const long long items = (long long)cfg.n_q_heads * cfg.head_dim;
  int nx = (int)((items + ct - 1) / ct);
  const long long score_loads = (long long)(n + 1) * cfg.n_q_heads;
  const int by_scores = (int)((score_loads + (long long)lg * ct - 1) / ((long long)lg * ct));
  if (p.do_evict && nx < by_scores) nx = by_scores;
  if (nx > cl_max) nx = cl_max;
  if (nx < 1) nx = 1;
  p.nx = nx;
  p.cand_per_cta = ((n + 1 + nx - 1) / nx + 3) / 4 * 4;   // a multiple of 4: 16-byte aligned blocks of logits
  set_combine_threads(p, ct);
}

// Pointers and launch geometry of one step of cache c for its current length.
void step_params(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos, float* out,
                 int32_t* evicted_pos, bool defer, StepParams& p) {
  const tova_config& cfg = c->cfg;
  const int n = c->len;
  unsigned char* base = c->base;
  p.K = base + c->lay.K;
  p.V = base + c->lay.V;
  p.pos = reinterpret_cast<int32_t*>(base + c->lay.pos);
  p.len = reinterpret_cast<int32_t*>(base + c->lay.len);
  p.logits = reinterpret_cast<float*>(base + c->lay.logits);
  p.part_ml = reinterpret_cast<float2*>(base + c->lay.part_ml);
  p.part_acc = reinterpret_cast<float*>(base + c->lay.part_acc);
  p.status = reinterpret_cast<int32_t*>(base + c->lay.status);
  p.cur_pos = reinterpret_cast<int32_t*>(base + c->lay.cur_pos);
  p.last_slot = reinterpret_cast<int32_t*>(base + c->lay.last_slot);
  p.q = q; p.k_new = k; p.v_new = v; p.out = out; p.evicted = evicted_pos; p.pos_t = pos;
  p.ld = c->lay.ld; p.pc = c->lay.pc;
  fill_geometry(p, cfg, n, c->chunk_rows, c->sm_count);
  p.scale2 = c->scale2;
  p.head_ml = reinterpret_cast<float2*>(base + c->lay.head_ml);
  p.policy = c->units > 0 ? tova::POLICY_TOVA : c->policy;
  p.keep_first = c->keep_first;
  // Head-wise policies write a different row in every KV head: no single "last written row" to fetch again,
  // so the streaming kernel requests its first tiles only after the dependency wait.
  if (c->units > 0) p.last_slot = nullptr;
  p.fuse_out = (c->fuse_merge && fused_merge_fits(cfg, c->chunk_rows, c->sm_count)) ? 1 : 0;
  p.merge_ctas = p.fuse_out ? (p.n_chunks + tova::SPLIT_MERGE_MAX_WARPS - 1) / tova::SPLIT_MERGE_MAX_WARPS : 1;
  if (p.merge_ctas < 1) p.merge_ctas = 1;
  if (c->poscomp_ws) {         // the rotating streaming kernel: partials through global memory, up to 4 heads per warp
    p.fuse_out = 0;
    p.merge_ctas = 1;
    p.hgroups = (p.G + tova::rope_unit_heads(p.G) - 1) / tova::rope_unit_heads(p.G);
  }
  if (p.fuse_out && defer) {   // the split kernel keeps copies of the new token's rows for the later insert
    p.k_stage = base + c->lay.df_k;
    p.v_stage = base + c->lay.df_v;
  }
}

int step_impl(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos, float* out,
              int32_t* evicted_pos, cudaStream_t st, bool allow_defer = true) {
  const tova_config& cfg = c->cfg;
  if (c->len >= cfg.capacity && !cfg.evict) return TOVA_ERR_FULL;
  if (c->shard_on) return TOVA_ERR_BAD_SHAPE;   // a sharded layer steps through its two-phase calls
  const bool defer = c->deferred && allow_defer && !c->poscomp_ws;
  StepParams p{};
  step_params(c, q, k, v, pos, out, evicted_pos, defer, p);
  cudaError_t e;
  if (cfg.dtype == TOVA_DTYPE_BF16) {
    e = cfg.head_dim == 128 ? launch_step<__nv_bfloat16, 128>(c, p, st, defer)
                            : launch_step<__nv_bfloat16, 64>(c, p, st, defer);
  } else {
    e = cfg.head_dim == 128 ? launch_step<float, 128>(c, p, st, defer) : launch_step<float, 64>(c, p, st, defer);
  }
  if (e != cudaSuccess) return TOVA_ERR_CUDA;
  if (c->len < cfg.capacity) c->len += 1;
  return TOVA_OK;
}

// Shortest run of prompt tokens worth the three launches of the bulk fill.
constexpr int BULK_FILL_MIN_TOKENS = 4;

template <int D>
cudaError_t launch_fill_d(tova_cache* c, const tova::FillParams& p, cudaStream_t st) {
  const size_t chunks = (size_t)p.F * p.B * p.Hkv * (D * 2 / 16);
  unsigned blocks = (unsigned)((chunks + 255) / 256);
  const unsigned cap_blocks = (unsigned)c->sm_count * 16u;
  if (blocks > cap_blocks) blocks = cap_blocks;
  if (blocks < 1) blocks = 1;
  tova::tova_fill_rows_kernel<D><<<blocks, 256, 0, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  c->launches += 1;
  if (p.out) {
    if (D == 128 && c->bulk_fill == 1) {
      constexpr size_t smem_tc = 64 * 1024 + 1024;
      static std::atomic<bool> configured_tc[64];
      if (c->device >= 0 && c->device < 64 && !configured_tc[c->device]) {
        e = cudaFuncSetAttribute(tova::tova_fill_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_tc);
        if (e != cudaSuccess) return e;
        configured_tc[c->device] = true;
      }
      dim3 grid((p.F + tova::FILLTC_Q_ROWS - 1) / tova::FILLTC_Q_ROWS, p.H, p.B);
      tova::tova_fill_attn_tc_kernel<<<grid, tova::FILLTC_THREADS, smem_tc, st>>>(p, c->fill_map_k, c->fill_map_v);
    } else {
      constexpr size_t smem = 4 * (size_t)tova::FILL_K_ROWS * D * 2 + 1024;
      static std::atomic<bool> configured[64];
      if (c->device >= 0 && c->device < 64 && !configured[c->device]) {
        e = cudaFuncSetAttribute(tova::tova_fill_attn_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        configured[c->device] = true;
      }
      dim3 grid((p.F + tova::FILL_Q_ROWS - 1) / tova::FILL_Q_ROWS, p.H, p.B);
      tova::tova_fill_attn_kernel<D><<<grid, tova::FILL_THREADS, smem, st>>>(p, c->fill_map_k, c->fill_map_v);
    }
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    c->launches += 1;
  }
  // A plain launch after the attention: a later split kernel, which starts fetching rows before its own
  // dependency wait, can then start only once the copies above have completed.
  tova::tova_fill_commit_kernel<<<(p.B + 127) / 128, 128, 0, st>>>(p);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  c->launches += 1;
  return cudaSuccess;
}

// F tokens into free rows of a bf16 state (len + F <= capacity): rows, positions, causal attention.
int launch_fill(tova_cache* c, const void* q, const void* k, const void* v, int F, int32_t first_pos, float* out,
                int32_t* evicted_pos, cudaStream_t st) {
  if (c->pending) {  // a deferred insert of an earlier token must land first
    if (cudaStreamWaitEvent(st, c->ev_join, 0) != cudaSuccess) return TOVA_ERR_CUDA;
    c->pending = false;
  }
  tova::FillParams p{};
  unsigned char* base = c->base;
  p.K = base + c->lay.K;
  p.V = base + c->lay.V;
  p.pos = reinterpret_cast<int32_t*>(base + c->lay.pos);
  p.len = reinterpret_cast<int32_t*>(base + c->lay.len);
  p.last_slot = reinterpret_cast<int32_t*>(base + c->lay.last_slot);
  p.cur_pos = reinterpret_cast<int32_t*>(base + c->lay.cur_pos);
  p.status = reinterpret_cast<int32_t*>(base + c->lay.status);
  p.q = q; p.k_new = k; p.v_new = v; p.out = out; p.evicted = evicted_pos;
  p.units = c->units > 1 ? c->units : 1;
  p.upos = c->units > 1 ? reinterpret_cast<int32_t*>(base + c->lay.upos) : nullptr;
  p.B = c->cfg.batch; p.H = c->cfg.n_q_heads; p.Hkv = c->cfg.n_kv_heads; p.G = p.H / p.Hkv;
  p.cap = c->cfg.capacity;
  p.n0 = c->len;
  p.F = F;
  p.first_pos = first_pos;
  p.scale2 = c->scale2;
  const cudaError_t e = c->cfg.head_dim == 128 ? launch_fill_d<128>(c, p, st) : launch_fill_d<64>(c, p, st);
  if (e != cudaSuccess) return TOVA_ERR_CUDA;
  c->len += F;
  return TOVA_OK;
}

// Fewest prompt tokens worth a chunk's five launches.
constexpr int CHUNK_MIN_TOKENS = 8;
constexpr size_t CHUNK_RESOLVE_SMEM_LIMIT = 200 * 1024;
constexpr size_t CHUNK_CLUSTER_SMEM_LIMIT = 216 * 1024;

inline size_t chunk_resolve_smem(const tova_config& cfg) {
  return sizeof(int32_t) * 2 * (size_t)cfg.capacity + sizeof(float) * (size_t)cfg.n_q_heads;
}

template <int D>
cudaError_t launch_chunk_d(tova_cache* c, const tova::ChunkParams& p, cudaStream_t st) {
  const unsigned cap_blocks = (unsigned)c->sm_count * 16u;
  auto blocks_for = [&](size_t items) {
    unsigned b = (unsigned)((items + 255) / 256);
    return b < 1 ? 1u : (b > cap_blocks ? cap_blocks : b);
  };
  cudaError_t e;
  tova::tova_chunk_stage_kernel<D><<<blocks_for((size_t)p.B * p.Hkv * tova::CHUNK_TOKENS * (D * 2 / 16)), 256, 0, st>>>(p);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  constexpr size_t smem = 4 * (size_t)tova::FILL_K_ROWS * D * 2 + 1024;
  static std::atomic<bool> configured[64];
  if (c->device >= 0 && c->device < 64 && !configured[c->device]) {
    if ((e = cudaFuncSetAttribute(tova::tova_chunk_attn_kernel<D, 0>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(tova::tova_chunk_attn_kernel<D, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(tova::tova_chunk_resolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  (int)CHUNK_RESOLVE_SMEM_LIMIT)) != cudaSuccess) return e;
    configured[c->device] = true;
  }
  const dim3 grid(p.H, p.B);
  tova::tova_chunk_attn_kernel<D, 0><<<grid, tova::FILL_THREADS, smem, st>>>(p, c->fill_map_k, c->fill_map_v, c->chunk_map_k,
                                                                         c->chunk_map_v);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  // The deletions: a cluster of CTAs per sequence with the logits staged in shared memory ahead of time, as
  // many CTAs as keep all sequences resident at once; one CTA per sequence reading global memory where
  // even one staged token does not fit.
  {
    int nc = tova::CHUNK_CLUSTER_MAX;
    while (nc > 1 && (long long)p.B * nc > c->sm_count) nc >>= 1;
    if (c->chunk_cluster > 0) nc = c->chunk_cluster;
    const int S = ((p.cap + nc - 1) / nc + 3) / 4 * 4;
    // Two or more tokens' logits staged: the kernel with one cluster barrier per token; one: the kernel with two.
    int nstage1 = tova::CHUNK_STAGES_MAX;
    while (nstage1 > 0 && tova::chunk_cluster1_smem(p.H, S, nstage1) > CHUNK_CLUSTER_SMEM_LIMIT) --nstage1;
    const bool one_barrier = nstage1 >= 2 && c->chunk_two_barriers == 0;
    int nstage = tova::CHUNK_STAGES_MAX;
    while (nstage > 0 && tova::chunk_cluster_smem(p.H, S, nstage) > CHUNK_CLUSTER_SMEM_LIMIT) --nstage;
    if (one_barrier) nstage = nstage1;
    if (nstage > 0 && c->chunk_cluster >= 0) {
      static std::atomic<bool> cl_configured[64];
      if (c->device >= 0 && c->device < 64 && !cl_configured[c->device]) {
        if ((e = cudaFuncSetAttribute(tova::tova_chunk_resolve_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)CHUNK_CLUSTER_SMEM_LIMIT)) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(tova::tova_chunk_resolve_cluster1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      (int)CHUNK_CLUSTER_SMEM_LIMIT)) != cudaSuccess) return e;
        cl_configured[c->device] = true;
      }
      cudaLaunchConfig_t cfg{};
      cfg.gridDim = dim3(nc, p.B);
      int nt = 256;                            // about one thread per candidate of a CTA
      while (nt < tova::CHUNK_CLUSTER_THREADS_MAX && nt < S + 1) nt *= 2;
      cfg.blockDim = dim3(nt);
      cfg.dynamicSmemBytes = one_barrier ? tova::chunk_cluster1_smem(p.H, S, nstage) : tova::chunk_cluster_smem(p.H, S, nstage);
      cfg.stream = st;
      cudaLaunchAttribute at[1];
      at[0].id = cudaLaunchAttributeClusterDimension;
      at[0].val.clusterDim.x = nc;
      at[0].val.clusterDim.y = 1;
      at[0].val.clusterDim.z = 1;
      cfg.attrs = at;
      cfg.numAttrs = 1;
      e = one_barrier ? cudaLaunchKernelEx(&cfg, tova::tova_chunk_resolve_cluster1_kernel, p, S, nstage)
                      : cudaLaunchKernelEx(&cfg, tova::tova_chunk_resolve_cluster_kernel, p, S, nstage);
    } else {
      tova::tova_chunk_resolve_kernel<<<p.B, tova::CHUNK_RESOLVE_THREADS, chunk_resolve_smem(c->cfg), st>>>(p);
      e = cudaGetLastError();
    }
    if (e != cudaSuccess) return e;
  }
  c->launches += 3;
  if (p.out) {
    tova::tova_chunk_attn_kernel<D, 1><<<grid, tova::FILL_THREADS, smem, st>>>(p, c->fill_map_k, c->fill_map_v, c->chunk_map_k,
                                                                           c->chunk_map_v);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    c->launches += 1;
  }
  tova::tova_chunk_scatter_kernel<D><<<blocks_for((size_t)p.B * p.cap * p.Hkv * (D * 2 / 16)), 256, 0, st>>>(p);
  if ((e = cudaGetLastError()) != cudaSuccess) return e;
  c->launches += 1;
  return cudaSuccess;
}

// C prompt tokens (CHUNK_MIN_TOKENS..64) onto a full bf16 state under the TOVA policy, through the caller's workspace.
int launch_chunk(tova_cache* c, const void* q, const void* k, const void* v, int C, int32_t first_pos, float* out,
                 int32_t* evicted_pos, cudaStream_t st) {
  if (c->pending) {
    if (cudaStreamWaitEvent(st, c->ev_join, 0) != cudaSuccess) return TOVA_ERR_CUDA;
    c->pending = false;
  }
  tova::ChunkParams p{};
  unsigned char* base = c->base;
  unsigned char* ws = c->chunk_ws;
  const ChunkLayout& L = c->chunk_lay;
  p.K = base + c->lay.K;
  p.V = base + c->lay.V;
  p.pos = reinterpret_cast<int32_t*>(base + c->lay.pos);
  p.cur_pos = reinterpret_cast<int32_t*>(base + c->lay.cur_pos);
  p.last_slot = reinterpret_cast<int32_t*>(base + c->lay.last_slot);
  p.status = reinterpret_cast<int32_t*>(base + c->lay.status);
  p.q = q; p.k_new = k; p.v_new = v; p.out = out; p.evicted = evicted_pos;
  p.Kst = ws + L.Kst;
  p.Vst = ws + L.Vst;
  p.lg = reinterpret_cast<float*>(ws + L.lg);
  p.rt = reinterpret_cast<float2*>(ws + L.rt);
  p.ml = reinterpret_cast<float2*>(ws + L.ml);
  p.death = reinterpret_cast<int32_t*>(ws + L.death);
  p.slot_token = reinterpret_cast<int32_t*>(ws + L.slot_token);
  p.first = reinterpret_cast<int32_t*>(ws + L.first);
  p.B = c->cfg.batch; p.H = c->cfg.n_q_heads; p.Hkv = c->cfg.n_kv_heads; p.G = p.H / p.Hkv;
  p.cap = c->cfg.capacity;
  p.ldc = L.ldc;
  p.capA = L.ldc - tova::CHUNK_TOKENS;
  p.C = C;
  p.first_pos = first_pos;
  p.keep_first = c->keep_first;
  p.window = c->policy == tova::POLICY_WINDOW ? 1 : 0;
  p.scale2 = c->scale2;
  const cudaError_t e = c->cfg.head_dim == 128 ? launch_chunk_d<128>(c, p, st) : launch_chunk_d<64>(c, p, st);
  return e == cudaSuccess ? TOVA_OK : TOVA_ERR_CUDA;
}

int check_step_args(const tova_cache* c, const void* q, const void* k, const void* v, const void* out) {
  if (!c || !q || !k || !v || !out) return TOVA_ERR_NULL;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return TOVA_ERR_ALIGN;
  return TOVA_OK;
}

}  // namespace

// Tiled view of a [B*Hkv*capacity, D] bf16 matrix for the tensor-core split
// kernel: boxes of 16 rows x 64 columns (128 bytes) with the 128-byte swizzle.
// The driver's encoder is looked up through the runtime, so the library has no
// link-time dependency on the driver.
int encode_state_map(CUtensorMap* map, void* base, const tova_config& cfg, int box_rows = tova::TILE_ROWS,
                     long long rows_per_head = 0) {
  typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static std::atomic<encode_fn> fn_cache{nullptr};
  encode_fn fn = fn_cache.load(std::memory_order_acquire);
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !sym)
      return TOVA_ERR_CUDA;
    fn = reinterpret_cast<encode_fn>(sym);
    fn_cache.store(fn, std::memory_order_release);
  }
  const cuuint64_t rows = (cuuint64_t)cfg.batch * cfg.n_kv_heads * (rows_per_head ? rows_per_head : cfg.capacity);
  const cuuint64_t dims[2] = {(cuuint64_t)cfg.head_dim, rows};
  const cuuint64_t strides[1] = {(cuuint64_t)cfg.head_dim * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? TOVA_OK : TOVA_ERR_CUDA;
}

// ---------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------
extern "C" {

size_t tova_cache_bytes(const tova_config* cfg) {
  int why;
  if (!config_ok(cfg, &why)) return 0;
  return make_layout(*cfg).total;
}

int tova_cache_init(tova_cache** out, const tova_config* cfg, void* dev_mem, size_t dev_bytes,
                    void* cuda_stream) {
  if (!out) return TOVA_ERR_NULL;
  *out = nullptr;
  int why;
  if (!config_ok(cfg, &why)) return why;
  if (!dev_mem) return TOVA_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(dev_mem) % ALIGN != 0) return TOVA_ERR_ALIGN;
  const Layout lay = make_layout(*cfg);
  if (dev_bytes < lay.total) return TOVA_ERR_WORKSPACE;

  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return TOVA_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TOVA_ERR_CUDA;

  tova_cache* c = new (std::nothrow) tova_cache();
  if (!c) return TOVA_ERR_CUDA;
  c->cfg = *cfg;
  if (c->cfg.sm_scale == 0.f) c->cfg.sm_scale = 1.f / std::sqrt((float)cfg->head_dim);
  c->lay = lay;
  c->base = static_cast<unsigned char*>(dev_mem);
  c->len = 0;
  c->launches = 0;
  c->sm_count = sms;
  c->device = dev;
  c->chunk_rows = pick_chunk_rows(*cfg, sms);
  if (c->chunk_rows < 0) { delete c; return TOVA_ERR_UNSUPPORTED; }
  c->scale2 = c->cfg.sm_scale * 1.4426950408889634f;
  c->elem = cfg->dtype == TOVA_DTYPE_BF16 ? 2 : 4;
  c->row_bytes = c->elem * cfg->head_dim;
  c->fuse_merge = true;
  c->policy = tova::POLICY_TOVA;
  c->keep_first = 0;
  c->units = 0;
  c->recent = 0;
  c->chunk_ws = nullptr;
  c->poscomp_ws = nullptr;
  c->shard_on = false;
  c->shard_scored = false;
  c->chunk_cluster = 0;
  c->chunk_two_barriers = 0;
  c->deferred = false;
  c->pending = false;
  c->side = nullptr;
  c->ev_fork = c->ev_join = nullptr;
  c->use_mma = wants_mma(*cfg);
  if (c->use_mma) {
    if ((long long)cfg->batch * cfg->n_kv_heads * cfg->capacity >= (1LL << 31)) { delete c; return TOVA_ERR_BAD_SHAPE; }
    if (encode_state_map(&c->map_k, c->base + lay.K, *cfg) != TOVA_OK ||
        encode_state_map(&c->map_v, c->base + lay.V, *cfg) != TOVA_OK) {
      delete c;
      return TOVA_ERR_CUDA;
    }
  }
  // Bulk fill of a prompt (bf16 states): tiled views in boxes of 64 rows.  Where they cannot be had
  // (a state of fewer rows than one box, 2^31 rows or more) prompts go token by token.
  c->bulk_fill = 1;
  c->fill_maps = false;
  {
    const long long rows = (long long)cfg->batch * cfg->n_kv_heads * cfg->capacity;
    if (cfg->dtype == TOVA_DTYPE_BF16 && rows >= tova::FILL_K_ROWS && rows < (1LL << 31))
      c->fill_maps = encode_state_map(&c->fill_map_k, c->base + lay.K, *cfg, tova::FILL_K_ROWS) == TOVA_OK &&
                     encode_state_map(&c->fill_map_v, c->base + lay.V, *cfg, tova::FILL_K_ROWS) == TOVA_OK;
  }

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // Rows that were never written are still read as part of 16-row tiles (their
  // weight is zero): they must hold finite numbers.
  const size_t kv_bytes = (size_t)cfg->batch * cfg->n_kv_heads * cfg->capacity * c->row_bytes;
  if (cudaMemsetAsync(c->base + lay.K, 0, kv_bytes, st) != cudaSuccess ||
      cudaMemsetAsync(c->base + lay.V, 0, kv_bytes, st) != cudaSuccess) {
    delete c;
    return TOVA_ERR_CUDA;
  }
  if (cudaMemsetAsync(c->base + lay.shard_words, 0, 8, st) != cudaSuccess) { delete c; return TOVA_ERR_CUDA; }
  // per-unit slot tables start at -1 (all bytes 0xff), accumulated scores at zero
  const size_t unit_bytes = (size_t)cfg->batch * cfg->n_kv_heads * cfg->capacity * 4;
  if (cudaMemsetAsync(c->base + lay.upos, 0xff, unit_bytes, st) != cudaSuccess ||
      cudaMemsetAsync(c->base + lay.uacc, 0, unit_bytes, st) != cudaSuccess ||
      cudaMemsetAsync(c->base + lay.uticket, 0, (size_t)cfg->batch * cfg->n_kv_heads * 4, st) != cudaSuccess) {
    delete c;
    return TOVA_ERR_CUDA;
  }
  const size_t n = (size_t)cfg->batch * cfg->capacity;
  const int threads = 256;
  const unsigned blocks = (unsigned)((n + threads - 1) / threads);
  tova::tova_init_kernel<<<blocks, threads, 0, st>>>(
      reinterpret_cast<int32_t*>(c->base + lay.pos), reinterpret_cast<int32_t*>(c->base + lay.len),
      reinterpret_cast<int32_t*>(c->base + lay.last_slot),
      reinterpret_cast<int32_t*>(c->base + lay.status),
      reinterpret_cast<int32_t*>(c->base + lay.cur_pos), cfg->batch, cfg->capacity);
  if (cudaGetLastError() != cudaSuccess) { delete c; return TOVA_ERR_CUDA; }
  c->launches += 1;
  *out = c;
  return TOVA_OK;
}

int tova_cache_set_chunk_rows(tova_cache* c, int32_t rows) {
  if (!c) return TOVA_ERR_NULL;
  if (rows == 0) { c->chunk_rows = pick_chunk_rows(c->cfg, c->sm_count); return TOVA_OK; }  // fits: init checked
  if (rows < tova::MIN_CHUNK_ROWS || rows > 8192 || rows % tova::MIN_CHUNK_ROWS != 0) return TOVA_ERR_BAD_SHAPE;
  const int chunks = (c->cfg.capacity + rows - 1) / rows;
  if (combine_smem_bound(c->cfg.n_q_heads, chunks + 1) > COMBINE_BASE_LIMIT) return TOVA_ERR_BAD_SHAPE;
  c->chunk_rows = rows;
  return TOVA_OK;
}

int tova_cache_set_policy(tova_cache* c, int32_t policy, int32_t arg) {
  if (!c) return TOVA_ERR_NULL;
  if (policy < TOVA_POLICY_TOVA || policy > TOVA_POLICY_H2O_HEAD) return TOVA_ERR_UNSUPPORTED;
  if (c->len != 0 || c->pending) return TOVA_ERR_BAD_SHAPE;   // the policy is fixed while the state is empty
  if (c->shard_on && policy != TOVA_POLICY_TOVA) return TOVA_ERR_UNSUPPORTED;   // the sharded step sums TOVA's weights
  if (policy == TOVA_POLICY_TOVA || policy == TOVA_POLICY_WINDOW) {
    // a droppable row must always exist, and Window compares ages that stay below the capacity only if the
    // state has been under this policy from the start
    if (arg < 0 || arg >= c->cfg.capacity) return TOVA_ERR_BAD_SHAPE;
    c->policy = policy == TOVA_POLICY_WINDOW ? tova::POLICY_WINDOW : tova::POLICY_TOVA;
    c->keep_first = arg;
    c->units = 0;
    return TOVA_OK;
  }
  if (c->poscomp_ws || c->shard_on) return TOVA_ERR_UNSUPPORTED;   // per-unit policies: not with compression or sharding
  if (policy == TOVA_POLICY_TOVA_HEAD) {
    if (arg != 0) return TOVA_ERR_BAD_SHAPE;
    c->policy = tova::POLICY_TOVA_HEAD;
    c->units = c->cfg.n_kv_heads;
    c->keep_first = 0;
    return TOVA_OK;
  }
  // H2O: arg = size of the recent window; 0 = the other half of the multi-state (Section 4.1)
  if (arg < 0 || arg > c->cfg.capacity) return TOVA_ERR_BAD_SHAPE;
  c->recent = arg ? arg : c->cfg.capacity - c->cfg.capacity / 2;
  c->policy = policy == TOVA_POLICY_H2O_LAYER ? tova::POLICY_H2O_LAYER : tova::POLICY_H2O_HEAD;
  c->units = policy == TOVA_POLICY_H2O_LAYER ? 1 : c->cfg.n_kv_heads;
  c->keep_first = 0;
  return TOVA_OK;
}

int tova_cache_set_bulk_prefill(tova_cache* c, int32_t on) {
  if (!c) return TOVA_ERR_NULL;
  if (on < 0 || on > 2) return TOVA_ERR_BAD_SHAPE;
  c->bulk_fill = on;
  return TOVA_OK;
}

namespace {
struct PosCompLayout { size_t table, q_rot, cpos, total; };
PosCompLayout make_poscomp_layout(const tova_config& c) {
  PosCompLayout L{};
  const size_t B = c.batch, H = c.n_q_heads, D = c.head_dim, cap = c.capacity;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.table = take(B * (cap + 1) * (D / 2) * 8);
  L.q_rot = take(B * H * D * 4);
  L.cpos = take(B * (cap + 1) * 8);
  L.total = off;
  return L;
}
}  // namespace

size_t tova_position_workspace_bytes(const tova_config* cfg) {
  int why;
  if (!config_ok(cfg, &why)) return 0;
  return make_poscomp_layout(*cfg).total;
}

int tova_cache_set_position_compression(tova_cache* c, void* dev_mem, size_t dev_bytes, float rope_base) {
  if (!c) return TOVA_ERR_NULL;
  if (c->len != 0 || c->pending) return TOVA_ERR_BAD_SHAPE;      // keys must be cached un-rotated from the first token
  if (!dev_mem) { c->poscomp_ws = nullptr; return TOVA_OK; }
  if (!(rope_base > 1.f) || !std::isfinite(rope_base)) return TOVA_ERR_BAD_SHAPE;
  if (c->units != 0 || c->shard_on || tova::poscomp_smem_bytes(c->cfg.capacity, c->cfg.head_dim) > POSCOMP_SMEM_LIMIT)
    return TOVA_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(dev_mem) % ALIGN != 0) return TOVA_ERR_ALIGN;
  const PosCompLayout L = make_poscomp_layout(c->cfg);
  if (dev_bytes < L.total) return TOVA_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(dev_mem);
  c->poscomp.table = reinterpret_cast<float2*>(ws + L.table);
  c->poscomp.q_rot = reinterpret_cast<float*>(ws + L.q_rot);
  c->poscomp.cpos = reinterpret_cast<double*>(ws + L.cpos);
  c->poscomp.rope_base = (double)rope_base;
  static_assert(sizeof(c->poscomp.inv_freq) / sizeof(double) >= 64, "table of inverse frequencies");
  if (c->cfg.head_dim > 128) return TOVA_ERR_UNSUPPORTED;
  for (int d = 0; d < c->cfg.head_dim / 2; ++d)
    c->poscomp.inv_freq[d] = std::pow((double)rope_base, -2.0 * (double)d / (double)c->cfg.head_dim);
  c->poscomp_ws = ws;
  return TOVA_OK;
}

int tova_cache_read_compressed_positions(const tova_cache* c, double* cpos, void* cuda_stream) {
  if (!c || !cpos) return TOVA_ERR_NULL;
  if (!c->poscomp_ws) return TOVA_ERR_UNSUPPORTED;
  const size_t bytes = (size_t)c->cfg.batch * (c->cfg.capacity + 1) * 8;
  return cudaMemcpyAsync(cpos, c->poscomp.cpos, bytes, cudaMemcpyDeviceToDevice, static_cast<cudaStream_t>(cuda_stream)) ==
                 cudaSuccess ? TOVA_OK : TOVA_ERR_CUDA;
}

size_t tova_shard_table_bytes(const tova_config* cfg, int32_t world) {
  int why;
  if (!config_ok(cfg, &why) || world < 1 || world > tova::SHARD_MAX_WORLD) return 0;
  return 2 * (size_t)world * cfg->batch * make_layout(*cfg).ld * sizeof(float);   // two halves, used alternately
}

int tova_cache_set_shard(tova_cache* c, int32_t rank, int32_t world, int32_t n_q_heads_total, void* const* peer_tables,
                         void* const* peer_flags) {
  if (!c) return TOVA_ERR_NULL;
  if (world < 1 || world > tova::SHARD_MAX_WORLD || rank < 0 || rank >= world || n_q_heads_total < c->cfg.n_q_heads)
    return TOVA_ERR_BAD_SHAPE;
  if (c->len != 0 || c->pending || !c->cfg.evict) return TOVA_ERR_BAD_SHAPE;
  if (c->units != 0 || c->policy != tova::POLICY_TOVA || c->poscomp_ws) return TOVA_ERR_UNSUPPORTED;   // layer-wise TOVA (with "+i")
  if (!peer_tables || !peer_tables[rank]) return TOVA_ERR_NULL;
  tova::ShardParams sp{};
  sp.rank = rank;
  sp.world = world;
  sp.h_total = n_q_heads_total;
  sp.tables = peer_flags ? world : 1;        // without flags the caller adds the ranks' vectors itself (a library all-reduce)
  for (int r = 0; r < world; ++r) {
    if (sp.tables > 1 && (!peer_tables[r] || !peer_flags[r])) return TOVA_ERR_NULL;
    sp.parts[r] = static_cast<float*>(peer_tables[sp.tables > 1 ? r : rank]);
    sp.flags[r] = sp.tables > 1 ? static_cast<int32_t*>(peer_flags[r]) : nullptr;
    if (!aligned16(sp.parts[r])) return TOVA_ERR_ALIGN;
  }
  sp.epoch = reinterpret_cast<int32_t*>(c->base + c->lay.shard_words);
  sp.ticket = sp.epoch + 1;
  c->shard = sp;
  c->shard_on = true;
  c->shard_scored = false;
  c->deferred = false;
  return TOVA_OK;
}

int tova_decode_step_scores(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos, float* out,
                            void* cuda_stream) {
  int rc = check_step_args(c, q, k, v, out);
  if (rc != TOVA_OK) return rc;
  if (!c->shard_on || c->shard_scored) return TOVA_ERR_BAD_SHAPE;   // not sharded, or a commit is outstanding
  StepParams p{};
  step_params(c, q, k, v, pos, out, nullptr, false, p);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  cudaError_t e;
  if (c->cfg.dtype == TOVA_DTYPE_BF16) {
    e = c->cfg.head_dim == 128 ? launch_step<__nv_bfloat16, 128>(c, p, st, false) : launch_step<__nv_bfloat16, 64>(c, p, st, false);
  } else {
    e = c->cfg.head_dim == 128 ? launch_step<float, 128>(c, p, st, false) : launch_step<float, 64>(c, p, st, false);
  }
  if (e != cudaSuccess) return TOVA_ERR_CUDA;
  c->shard_scored = true;
  return TOVA_OK;
}

int tova_decode_step_commit(tova_cache* c, const void* k, const void* v, int32_t* evicted_pos, void* cuda_stream) {
  if (!c || !k || !v) return TOVA_ERR_NULL;
  if (!aligned16(k) || !aligned16(v)) return TOVA_ERR_ALIGN;
  if (!c->shard_on || !c->shard_scored) return TOVA_ERR_BAD_SHAPE;
  StepParams p{};
  step_params(c, nullptr, k, v, 0, nullptr, evicted_pos, false, p);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (c->cfg.dtype == TOVA_DTYPE_BF16) {
    if (c->cfg.head_dim == 128) tova::tova_shard_commit_kernel<__nv_bfloat16, 128><<<p.B, tova::SHARD_THREADS, 0, st>>>(p, c->shard);
    else tova::tova_shard_commit_kernel<__nv_bfloat16, 64><<<p.B, tova::SHARD_THREADS, 0, st>>>(p, c->shard);
  } else {
    if (c->cfg.head_dim == 128) tova::tova_shard_commit_kernel<float, 128><<<p.B, tova::SHARD_THREADS, 0, st>>>(p, c->shard);
    else tova::tova_shard_commit_kernel<float, 64><<<p.B, tova::SHARD_THREADS, 0, st>>>(p, c->shard);
  }
  if (cudaGetLastError() != cudaSuccess) return TOVA_ERR_CUDA;
  c->launches += 1;
  c->shard_scored = false;
  if (c->len < c->cfg.capacity) c->len += 1;
  return TOVA_OK;
}

int tova_cache_set_chunk_cluster(tova_cache* c, int32_t ctas) {
  if (!c) return TOVA_ERR_NULL;
  if (ctas != -1 && ctas != 0 && ctas != 1 && ctas != 2 && ctas != 4 && ctas != 8) return TOVA_ERR_BAD_SHAPE;
  c->chunk_cluster = ctas;
  return TOVA_OK;
}

int tova_cache_set_chunk_barriers(tova_cache* c, int32_t per_token) {
  if (!c) return TOVA_ERR_NULL;
  if (per_token != 0 && per_token != 2) return TOVA_ERR_BAD_SHAPE;
  c->chunk_two_barriers = per_token == 2 ? 1 : 0;
  return TOVA_OK;
}

int tova_cache_set_fused_merge(tova_cache* c, int32_t on) {
  if (!c) return TOVA_ERR_NULL;
  c->fuse_merge = on != 0;
  return TOVA_OK;
}

int tova_decode_step(tova_cache* c, const void* q, const void* k, const void* v, int32_t pos, float* out,
                     int32_t* evicted_pos, void* cuda_stream) {
  int rc = check_step_args(c, q, k, v, out);
  if (rc != TOVA_OK) return rc;
  return step_impl(c, q, k, v, pos, out, evicted_pos, static_cast<cudaStream_t>(cuda_stream));
}

int tova_prefill(tova_cache* c, const void* q, const void* k, const void* v, int32_t n_tokens,
                 int32_t first_pos, float* out, int32_t* evicted_pos, void* cuda_stream) {
  if (!c) return TOVA_ERR_NULL;
  if (n_tokens < 0 || c->shard_on) return TOVA_ERR_BAD_SHAPE;   // a sharded layer steps through its two-phase calls
  if (n_tokens == 0) return TOVA_OK;
  float* scratch_out = reinterpret_cast<float*>(c->base + c->lay.st_out);
  int rc = check_step_args(c, q, k, v, out ? (const void*)out : (const void*)scratch_out);
  if (rc != TOVA_OK) return rc;
  if (!c->cfg.evict && (int64_t)c->len + n_tokens > c->cfg.capacity) return TOVA_ERR_FULL;
  const size_t B = c->cfg.batch, H = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
  const size_t q_stride = B * H * D * c->elem, kv_stride = B * Hkv * D * c->elem;
  int32_t done = 0;
  // Tokens that fit into free rows are not followed by a deletion (g(t) = min(t, k), Section 3.3):
  // they are ordinary causal attention and go through the bulk kernels in one piece.
  {
    const int room = c->cfg.capacity - c->len;
    const int F = n_tokens < room ? n_tokens : room;
    // (H2O accumulates scores from the first token on: token by token; head-wise TOVA only needs its slot tables)
    const bool unit_ok = c->units == 0 || c->policy == tova::POLICY_TOVA_HEAD;
    if (c->bulk_fill && c->fill_maps && F >= BULK_FILL_MIN_TOKENS && unit_ok && !c->poscomp_ws) {
      rc = launch_fill(c, q, k, v, F, first_pos, out, evicted_pos, static_cast<cudaStream_t>(cuda_stream));
      if (rc != TOVA_OK) return rc;
      done = F;
    }
  }
  // Tokens that meet a full state: chunks of up to 64 through the caller's workspace, where one was given
  // (TOVA or Window, with or without protected first positions; bf16 states).
  const bool chunked = c->chunk_ws && c->bulk_fill && c->cfg.evict && c->units == 0 &&
                       (c->policy == tova::POLICY_TOVA || c->policy == tova::POLICY_WINDOW) && !c->poscomp_ws;
  for (int32_t t = done; t < n_tokens;) {
    if (chunked && c->len == c->cfg.capacity && n_tokens - t >= CHUNK_MIN_TOKENS) {
      const int C = n_tokens - t < tova::CHUNK_TOKENS ? n_tokens - t : tova::CHUNK_TOKENS;
      rc = launch_chunk(c, static_cast<const unsigned char*>(q) + t * q_stride,
                        static_cast<const unsigned char*>(k) + t * kv_stride,
                        static_cast<const unsigned char*>(v) + t * kv_stride, C,
                        first_pos < 0 ? first_pos : first_pos + t, out ? out + (size_t)t * B * H * D : nullptr,
                        evicted_pos ? evicted_pos + (size_t)t * B : nullptr, static_cast<cudaStream_t>(cuda_stream));
      if (rc != TOVA_OK) return rc;
      t += C;
      continue;
    }
    rc = step_impl(c, static_cast<const unsigned char*>(q) + t * q_stride,
                   static_cast<const unsigned char*>(k) + t * kv_stride,
                   static_cast<const unsigned char*>(v) + t * kv_stride,
                   first_pos < 0 ? first_pos : first_pos + t,
                   out ? out + (size_t)t * B * H * D : scratch_out,
                   evicted_pos ? evicted_pos + (size_t)t * B * (c->units > 0 ? c->units : 1) : nullptr,
                   static_cast<cudaStream_t>(cuda_stream),
                   /*allow_defer=*/false);  // consecutive tokens of one cache cannot overlap anyway
    if (rc != TOVA_OK) return rc;
    ++t;
  }
  return TOVA_OK;
}

size_t tova_prefill_workspace_bytes(const tova_config* cfg) {
  int why;
  if (!config_ok(cfg, &why) || cfg->dtype != TOVA_DTYPE_BF16) return 0;
  return make_chunk_layout(*cfg).total;
}

int tova_cache_set_prefill_workspace(tova_cache* c, void* dev_mem, size_t dev_bytes) {
  if (!c) return TOVA_ERR_NULL;
  if (!dev_mem) { c->chunk_ws = nullptr; return TOVA_OK; }      // back to token-by-token
  if (c->cfg.dtype != TOVA_DTYPE_BF16 || !c->fill_maps || chunk_resolve_smem(c->cfg) > CHUNK_RESOLVE_SMEM_LIMIT)
    return TOVA_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(dev_mem) % ALIGN != 0) return TOVA_ERR_ALIGN;
  const ChunkLayout L = make_chunk_layout(c->cfg);
  if (dev_bytes < L.total) return TOVA_ERR_WORKSPACE;
  unsigned char* ws = static_cast<unsigned char*>(dev_mem);
  if (encode_state_map(&c->chunk_map_k, ws + L.Kst, c->cfg, tova::FILL_K_ROWS, tova::CHUNK_TOKENS) != TOVA_OK ||
      encode_state_map(&c->chunk_map_v, ws + L.Vst, c->cfg, tova::FILL_K_ROWS, tova::CHUNK_TOKENS) != TOVA_OK)
    return TOVA_ERR_CUDA;
  c->chunk_lay = L;
  c->chunk_ws = ws;
  return TOVA_OK;
}

namespace {
// The address under which the GPU can read or write a host buffer in place:
// page-locked (pinned or registered) memory only; null for pageable memory.
void* device_view_of_host(const void* host) {
  cudaPointerAttributes a{};
  if (cudaPointerGetAttributes(&a, host) != cudaSuccess) {
    (void)cudaGetLastError();   // older runtimes report pageable memory as an error: clear it
    return nullptr;
  }
  if (a.type != cudaMemoryTypeHost || !a.devicePointer || !aligned16(a.devicePointer)) return nullptr;
  return a.devicePointer;
}
}  // namespace

int tova_decode_step_host(tova_cache* c, const void* q_host, const void* k_host, const void* v_host,
                          int32_t pos, float* out_host, int32_t* evicted_pos_host, void* cuda_stream) {
  if (!c || !q_host || !k_host || !v_host || !out_host) return TOVA_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  // Page-locked buffers: no copy calls; five small copies per step would cost more than the step.
  {
    void* dq = device_view_of_host(q_host);
    void* dk = device_view_of_host(k_host);
    void* dv = device_view_of_host(v_host);
    void* dout = device_view_of_host(out_host);
    void* dev_ev = evicted_pos_host ? device_view_of_host(evicted_pos_host) : nullptr;
    if (dq && dk && dv && dout && (dev_ev || !evicted_pos_host)) {
      const size_t B = c->cfg.batch, H = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
      const int nq = (int)(B * H * D * c->elem / 16), nk = (int)(B * Hkv * D * c->elem / 16);
      unsigned char* base = c->base;
      const int threads = 256;
      int blocks = (nq + 2 * nk + threads - 1) / threads;
      if (blocks > 4 * c->sm_count) blocks = 4 * c->sm_count;
      // Every output element is written once, in place.  The inputs are read in place too while few warps
      // share a head group's q (each reads it over the bus: measured faster up to 8 chunks per group);
      // beyond that one small kernel brings q, k, v across once.
      const void *sq = dq, *sk = dk, *sv = dv;
      if ((c->cfg.capacity + c->chunk_rows - 1) / c->chunk_rows > tova::SPLIT_MERGE_MAX_WARPS) {
        tova::tova_fetch_inputs_kernel<<<blocks, threads, 0, st>>>(
            reinterpret_cast<uint4*>(base + c->lay.st_q), static_cast<const uint4*>(dq), nq,
            reinterpret_cast<uint4*>(base + c->lay.st_k), static_cast<const uint4*>(dk),
            reinterpret_cast<uint4*>(base + c->lay.st_v), static_cast<const uint4*>(dv), nk);
        if (cudaGetLastError() != cudaSuccess) return TOVA_ERR_CUDA;
        c->launches += 1;
        sq = base + c->lay.st_q; sk = base + c->lay.st_k; sv = base + c->lay.st_v;
      }
      int rc = step_impl(c, sq, sk, sv, pos, static_cast<float*>(dout), static_cast<int32_t*>(dev_ev), st,
                         /*allow_defer=*/false);
      if (rc != TOVA_OK) return rc;
      return cudaStreamSynchronize(st) == cudaSuccess ? TOVA_OK : TOVA_ERR_CUDA;
    }
  }
  const size_t B = c->cfg.batch, H = c->cfg.n_q_heads, Hkv = c->cfg.n_kv_heads, D = c->cfg.head_dim;
  const size_t qb = B * H * D * c->elem, kb = B * Hkv * D * c->elem, ob = B * H * D * sizeof(float);
  unsigned char* base = c->base;
  if (cudaMemcpyAsync(base + c->lay.st_q, q_host, qb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(base + c->lay.st_k, k_host, kb, cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(base + c->lay.st_v, v_host, kb, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return TOVA_ERR_CUDA;
  int rc = step_impl(c, base + c->lay.st_q, base + c->lay.st_k, base + c->lay.st_v, pos,
                     reinterpret_cast<float*>(base + c->lay.st_out),
                     reinterpret_cast<int32_t*>(base + c->lay.st_ev), st, /*allow_defer=*/false);
  if (rc != TOVA_OK) return rc;
  if (cudaMemcpyAsync(out_host, base + c->lay.st_out, ob, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TOVA_ERR_CUDA;
  if (evicted_pos_host &&
      cudaMemcpyAsync(evicted_pos_host, base + c->lay.st_ev, B * (c->units > 0 ? c->units : 1) * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return TOVA_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return TOVA_ERR_CUDA;
  return TOVA_OK;
}

int tova_cache_join(tova_cache* c, void* cuda_stream) {
  if (!c) return TOVA_ERR_NULL;
  if (c->pending) {
    if (cudaStreamWaitEvent(static_cast<cudaStream_t>(cuda_stream), c->ev_join, 0) != cudaSuccess)
      return TOVA_ERR_CUDA;
    c->pending = false;
  }
  return TOVA_OK;
}

int tova_cache_set_deferred_eviction(tova_cache* c, int32_t on) {
  if (!c) return TOVA_ERR_NULL;
  if (on && !c->side) {
    if (cudaStreamCreateWithFlags(&c->side, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&c->ev_join, cudaEventDisableTiming) != cudaSuccess)
      return TOVA_ERR_CUDA;
  }
  if (!on && c->pending) return TOVA_ERR_BAD_SHAPE;  // join first
  c->deferred = on != 0;
  return TOVA_OK;
}

int tova_cache_read(const tova_cache* c_in, int32_t* len, int32_t* positions, void* k_out, void* v_out,
                    int32_t* status, void* cuda_stream) {
  if (!c_in) return TOVA_ERR_NULL;
  tova_cache* c = const_cast<tova_cache*>(c_in);  // joining a deferred eviction updates host bookkeeping only
  if (tova_cache_join(c, cuda_stream) != TOVA_OK) return TOVA_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t B = c->cfg.batch, Hkv = c->cfg.n_kv_heads, cap = c->cfg.capacity;
  const size_t kvb = B * Hkv * cap * c->row_bytes;
  const unsigned char* base = c->base;
  bool ok = true;
  if (len) ok &= cudaMemcpyAsync(len, base + c->lay.len, B * 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (positions) {
    const bool per_head = c->units > 1;     // head-wise policies: one slot table per KV head
    ok &= cudaMemcpyAsync(positions, base + (per_head ? c->lay.upos : c->lay.pos), B * (per_head ? Hkv : 1) * cap * 4,
                          cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  }
  if (k_out) ok &= cudaMemcpyAsync(k_out, base + c->lay.K, kvb, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (v_out) ok &= cudaMemcpyAsync(v_out, base + c->lay.V, kvb, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  if (status) ok &= cudaMemcpyAsync(status, base + c->lay.status, 4, cudaMemcpyDeviceToDevice, st) == cudaSuccess;
  return ok ? TOVA_OK : TOVA_ERR_CUDA;
}

int tova_cache_read_scores(const tova_cache* c, float* scores, void* cuda_stream) {
  if (!c || !scores) return TOVA_ERR_NULL;
  if (c->policy != tova::POLICY_H2O_LAYER && c->policy != tova::POLICY_H2O_HEAD) return TOVA_ERR_UNSUPPORTED;
  const size_t bytes = (size_t)c->cfg.batch * c->units * c->cfg.capacity * 4;
  return cudaMemcpyAsync(scores, c->base + c->lay.uacc, bytes, cudaMemcpyDeviceToDevice,
                         static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? TOVA_OK : TOVA_ERR_CUDA;
}

int32_t tova_cache_units(const tova_cache* c) { return c ? (c->units > 0 ? c->units : 1) : -1; }

int32_t tova_cache_len(const tova_cache* c) { return c ? c->len : -1; }
int64_t tova_cache_launches(const tova_cache* c) { return c ? c->launches : -1; }

int tova_cache_destroy(tova_cache* c) {
  if (!c) return TOVA_ERR_NULL;
  if (c->side) {
    cudaStreamSynchronize(c->side);
    cudaEventDestroy(c->ev_fork);
    cudaEventDestroy(c->ev_join);
    cudaStreamDestroy(c->side);
  }
  delete c;
  return TOVA_OK;
}

const char* tova_strerror(int status) {
  switch (status) {
    case TOVA_OK: return "ok";
    case TOVA_ERR_NULL: return "a required pointer is NULL";
    case TOVA_ERR_BAD_SHAPE: return "shape or size out of range";
    case TOVA_ERR_UNSUPPORTED: return "unsupported head_dim or dtype";
    case TOVA_ERR_ALIGN: return "pointer not aligned as required";
    case TOVA_ERR_WORKSPACE: return "device block smaller than tova_cache_bytes()";
    case TOVA_ERR_FULL: return "state is full and eviction is off";
    case TOVA_ERR_CUDA: return "CUDA runtime call or kernel launch failed";
    case TOVA_ERR_DEVICE: return "a device-side check failed";
    case TOVA_ERR_STATIC_LIMIT:
      return "this shape needs more scratch than the library's built-in 8 MiB array holds";
    default: return "unknown status";
  }
}

}  // extern "C"

// ---------------------------------------------------------------------------
// A decode step for callers that cannot allocate device memory.
// ---------------------------------------------------------------------------
// The scratch the two kernels exchange (logits, chunk partials, per-block
// minima, tickets, status words) normally lives in the block the caller
// allocates for tova_cache_init.  Here it lives in an array that is part of the
// loaded module, so the call needs no workspace from anybody.  Every device
// context that loads the library carries these bytes until it exits.
namespace {

constexpr size_t STATIC_SCRATCH_BYTES = (size_t)TOVA_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

struct StaticDevice {
  std::atomic<bool> ready{false};
  unsigned char* scratch = nullptr;  // device address of g_static_scratch on this device
  int sm_count = 0;
};
StaticDevice g_static_dev[64];
std::mutex g_static_setup;   // first calls from several host threads: one of them does the look-up

struct StaticLayout {
  size_t logits, part_ml, part_acc, control, total;
  int ld, pc;
};

StaticLayout make_static_layout(const tova_config& c, int chunk_rows) {
  StaticLayout L{};
  const size_t B = c.batch, H = c.n_q_heads, D = c.head_dim, cap = c.capacity;
  L.ld = (int)((cap + 1 + 3) / 4 * 4);
  L.pc = (int)((cap + chunk_rows - 1) / chunk_rows) + 1;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
  L.control = take(B * 4 /*len*/ + 8 /*status, cur_pos*/);
  L.logits = take(B * H * L.ld * 4);
  L.part_ml = take(B * H * L.pc * 8);
  L.part_acc = take(B * H * (size_t)(L.pc - 1) * D * 4);
  L.total = off;
  return L;
}

}  // namespace

extern "C" int tova_decode_step_static(const tova_config* cfg, void* K, void* V, int32_t* positions,
                                       int32_t n_live, const void* q, const void* k, const void* v,
                                       int32_t pos, float* out, int32_t* evicted_pos, int32_t* status,
                                       void* cuda_stream) {
  int why;
  if (!config_ok(cfg, &why)) return why;
  if (!K || !V || !positions || !q || !k || !v || !out) return TOVA_ERR_NULL;
  if (!aligned16(K) || !aligned16(V) || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
    return TOVA_ERR_ALIGN;
  if (n_live < 0 || n_live > cfg->capacity || pos < 0) return TOVA_ERR_BAD_SHAPE;
  if (n_live == cfg->capacity && !cfg->evict) return TOVA_ERR_FULL;

  // One-time set-up per device, with that device current: the array's name is
  // only a host-side handle, kernels need the address the runtime reports.
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return TOVA_ERR_CUDA;
  StaticDevice& sd = g_static_dev[dev];
  if (!sd.ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> guard(g_static_setup);
    if (!sd.ready.load(std::memory_order_relaxed)) {
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return TOVA_ERR_CUDA;
      int sms = 0;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TOVA_ERR_CUDA;
      sd.scratch = static_cast<unsigned char*>(ptr);
      sd.sm_count = sms;
      sd.ready.store(true, std::memory_order_release);
    }
  }

  const int chunk_rows = pick_chunk_rows(*cfg, sd.sm_count);
  if (chunk_rows < 0) return TOVA_ERR_UNSUPPORTED;
  const StaticLayout lay = make_static_layout(*cfg, chunk_rows);
  if (lay.total > STATIC_SCRATCH_BYTES) return TOVA_ERR_STATIC_LIMIT;

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  unsigned char* base = sd.scratch;
  const size_t B = cfg->batch;
  // The status word must start at zero; the array keeps the previous call's contents.  A caller that
  // wants to see a failed device-side check passes its own word, which is cleared the same way.
  if (cudaMemsetAsync(base + lay.control, 0, B * 4 + 8, st) != cudaSuccess) return TOVA_ERR_CUDA;
  if (status && cudaMemsetAsync(status, 0, 4, st) != cudaSuccess) return TOVA_ERR_CUDA;

  StepParams p{};
  p.K = K;
  p.V = V;
  p.pos = positions;
  p.len = reinterpret_cast<int32_t*>(base + lay.control);
  p.cur_pos = reinterpret_cast<int32_t*>(base + lay.control + B * 4) + 1;
  p.status = status ? status : p.cur_pos - 1;
  p.logits = reinterpret_cast<float*>(base + lay.logits);
  p.part_ml = reinterpret_cast<float2*>(base + lay.part_ml);
  p.part_acc = reinterpret_cast<float*>(base + lay.part_acc);
  p.q = q; p.k_new = k; p.v_new = v; p.out = out; p.evicted = evicted_pos; p.pos_t = pos;
  p.ld = lay.ld; p.pc = lay.pc;
  fill_geometry(p, *cfg, n_live, chunk_rows, sd.sm_count);
  const float scale = cfg->sm_scale == 0.f ? 1.f / std::sqrt((float)cfg->head_dim) : cfg->sm_scale;
  p.scale2 = scale * 1.4426950408889634f;

  tova_cache shim{};  // launch_step reads the device, the tensor maps and counts launches
  shim.device = dev;
  shim.sm_count = sd.sm_count;
  shim.use_mma = wants_mma(*cfg);
  if (shim.use_mma) {
    if ((long long)cfg->batch * cfg->n_kv_heads * cfg->capacity >= (1LL << 31)) return TOVA_ERR_BAD_SHAPE;
    if (encode_state_map(&shim.map_k, K, *cfg) != TOVA_OK || encode_state_map(&shim.map_v, V, *cfg) != TOVA_OK)
      return TOVA_ERR_CUDA;
  }
  cudaError_t e;
  if (cfg->dtype == TOVA_DTYPE_BF16) {
    e = cfg->head_dim == 128 ? launch_step<__nv_bfloat16, 128>(&shim, p, st, false)
                             : launch_step<__nv_bfloat16, 64>(&shim, p, st, false);
  } else {
    e = cfg->head_dim == 128 ? launch_step<float, 128>(&shim, p, st, false)
                             : launch_step<float, 64>(&shim, p, st, false);
  }
  return e == cudaSuccess ? TOVA_OK : TOVA_ERR_CUDA;
}
