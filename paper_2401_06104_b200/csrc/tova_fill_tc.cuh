// Causal attention of a prompt run on the 5th-generation tensor cores (sm_100a): the same
// operation as tova_fill_attn_kernel (tova_fill.cuh; Eq. 6-7 while the state has free rows),
// with both contractions issued as tcgen05.mma from shared-memory descriptors and their
// accumulators in tensor memory (TMEM).
//
// One CTA per (128 query tokens, query head, sequence): 256 soft-max threads - query row i = TMEM lane i, shared
// by two threads (warps w and w + 4), each taking half of a tile's logits and half of O's columns - and one more
// warp whose first lane issues every copy and every contraction.  Per tile of 64 state rows:
//   TMA (tiled, 128-byte swizzle)  K tile, V tile -> shared memory (one buffer each; the next tile is requested
//                as soon as the contraction that read the buffer is complete)
//   tcgen05.mma  S[128 x 64]  = Q[128 x D] . K^T          (A, B K-major; fp32 in TMEM, two S buffers: S of tile
//                i+1 is issued as soon as its K tile is there, ahead of O += P V of tile i)
//   tcgen05.ld   half a row of S -> registers (row maxima of the two halves exchanged through shared memory at the
//                barrier the two warps of a row share); the weights of the thread's half; online soft-max in the base-2 domain; weights as hi + lo
//                bf16 terms -> tcgen05.st back into the tile's S buffer, where they are the A operand of the
//                second contraction (no trip through shared memory); if a row's running max moved, O is
//                rescaled in TMEM (tcgen05.ld / tcgen05.st)
//   tcgen05.mma  O[128 x D] += P_hi . V + P_lo . V         (A in tensor memory, B = V tile as stored, MN-major)
// The roles meet through mbarriers only (tcgen05.commit for the contractions, 256 arrivals for a tile's weights):
// the soft-max of tile i+1 runs while the tensor cores work on O += P V of tile i, and only writing the new
// weights and touching O wait for that contraction.  Two CTAs share an SM (65 KiB of shared memory, 256 of the
// 512 TMEM columns each).  Every wait is bounded; a wait that runs out sets the status word, the roles drain
// through their own bounded waits, and the CTA still frees its TMEM.
#pragma once

#include "tova_fill.cuh"

namespace tova {

constexpr int FILLTC_Q_ROWS = 128;
constexpr int FILLTC_SOFTMAX_THREADS = 256;   // two threads per query row: each takes half of a tile's 64 logits, half of O's columns
constexpr int FILLTC_THREADS = FILLTC_SOFTMAX_THREADS + 32;   // plus one warp whose first lane issues copies and contractions
constexpr int FILLTC_TMEM_COLS = 256;   // S of even and odd tiles: 64 columns each, O: 128 columns

// Shared-memory matrix descriptor: start address, leading / stride byte offsets (units of 16 bytes),
// descriptor version 1 (sm_100), 128-byte swizzle.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

// Instruction descriptor of kind::f16: fp32 accumulator, bf16 A and B, A K-major, B K-major or MN-major.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int M, int N, bool b_mn_major) {
  uint32_t d = 0;
  d |= 1u << 4;                        // D format: f32
  d |= 1u << 7;                        // A format: bf16
  d |= 1u << 10;                       // B format: bf16
  d |= (b_mn_major ? 1u : 0u) << 16;   // B major
  d |= (uint32_t)(N >> 3) << 17;
  d |= (uint32_t)(M >> 4) << 24;
  return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The same with the A operand in tensor memory: row i of A in TMEM lane i, its K elements packed two per 32-bit
// column from a_tmem on.
__device__ __forceinline__ void umma_bf16_a_tmem(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}

// The mbarrier receives one arrival once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_addr(bar))
               : "memory");
}

// One arrival of this thread on an mbarrier of its own CTA.
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// Barrier `id` (1..15) among `count` threads of the CTA (a multiple of 32; whole warps take part).
__device__ __forceinline__ void named_barrier_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}

// Bounded wait of the fill kernel (two seconds, as everywhere).
__device__ __forceinline__ bool fill_wait(uint64_t* bar, uint32_t parity) { return mbar_wait_bounded(bar, parity); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 2^x, hardware approximation (relative error about 2^-22; -inf gives 0; results below 2^-126 flush to 0).
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Two fp32 operations in one instruction (sm_100: packed operands in a 64-bit register).
__device__ __forceinline__ uint64_t pack_f2(float lo, float hi) {
  uint64_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f2(uint64_t v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t fma_f2(uint64_t a, uint64_t b, uint64_t c) {
  uint64_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ uint64_t add_f2(uint64_t a, uint64_t b) {
  uint64_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

// 32 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])),
        "r"(__float_as_uint(v[3])), "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])),
        "r"(__float_as_uint(v[7])), "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])),
        "r"(__float_as_uint(v[11])), "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])),
        "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])), "r"(__float_as_uint(v[16])),
        "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
        "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])),
        "r"(__float_as_uint(v[23])), "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])),
        "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])), "r"(__float_as_uint(v[28])),
        "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
// 16 consecutive 32-bit columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]),
        "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// grid = (ceil(F/128), H, B), block = 288.  Dynamic shared memory: Q (32 KiB) + K, V tiles (16 KiB each) + 1 KiB
// alignment slack.  head_dim 128 only.
__global__ void __launch_bounds__(FILLTC_THREADS, 2)
    tova_fill_attn_tc_kernel(const FillParams p, const __grid_constant__ CUtensorMap map_k,
                             const __grid_constant__ CUtensorMap map_v) {
  constexpr int D = 128;
  constexpr int KT = FILL_K_ROWS;                 // 64 state rows per tile
  constexpr int Q_BYTES = FILLTC_Q_ROWS * D * 2;  // two boxes of [128 rows][128 bytes]
  constexpr int T_BYTES = KT * D * 2;             // two boxes of [64 rows][128 bytes]

  extern __shared__ unsigned char filltc_smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(filltc_smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char* q_s = smem;
  unsigned char* k_s = q_s + Q_BYTES;
  unsigned char* v_s = k_s + T_BYTES;
  // K tile, V tile landed; S = Q K^T, O += P V completed (tcgen05.commit); weights of a tile written (256 arrivals)
  // (one S barrier per S buffer: a barrier then completes once per two tiles, and a waiter can never be two phases behind)
  __shared__ __align__(8) uint64_t bar_k, bar_v, bar_s[2], bar_o, bar_p;
  __shared__ uint32_t tmem_base_s;
  __shared__ float half_sum[2][FILLTC_Q_ROWS];   // the two halves of a row add up their sums at the end
  __shared__ float half_max[2][2][FILLTC_Q_ROWS];   // ... and exchange their tile maxima (double-buffered by tile)

  // A wait that ran out anywhere in this launch (or before) has left its code: the roles of that block have lost
  // each other, and the blocks still to come give up at once instead of each waiting out its own limit.
  if (*reinterpret_cast<volatile int32_t*>(p.status) != 0) return;

  const int tid = threadIdx.x, warp = tid >> 5;
  const int tile_q = gridDim.x - 1 - blockIdx.x;          // longest rows first
  const int t0 = tile_q * FILLTC_Q_ROWS;
  const int h = blockIdx.y, b = blockIdx.z;
  const int kvh = h / p.G;
  const int head_row0 = (b * p.Hkv + kvh) * p.cap;
  const int t_last = min(t0 + FILLTC_Q_ROWS, p.F) - 1;
  const int n_keys = p.n0 + t_last + 1;
  const int n_tiles = (n_keys + KT - 1) / KT;

  if (tid == 0) {
    mbar_init(&bar_k, 1);
    mbar_init(&bar_v, 1);
    mbar_init(&bar_s[0], 1);
    mbar_init(&bar_s[1], 1);
    mbar_init(&bar_o, 1);
    mbar_init(&bar_p, FILLTC_SOFTMAX_THREADS);
    mbar_fence_init();
  }
  if (warp == 0) {   // one warp allocates the CTA's tensor memory and gives up the right to allocate more
    __syncwarp();
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&tmem_base_s)),
                 "r"(FILLTC_TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Q tile -> shared memory, K-major with the 128-byte swizzle; rows past the run repeat its last token.
  {
    const __nv_bfloat16* qg = static_cast<const __nv_bfloat16*>(p.q);
    for (int i = tid; i < FILLTC_Q_ROWS * (D / 8); i += FILLTC_THREADS) {
      const int r = i / (D / 8), ch = i % (D / 8);
      const int t = min(t0 + r, p.F - 1);
      const uint4 w = *reinterpret_cast<const uint4*>(qg + (((size_t)t * p.B + b) * p.H + h) * D + ch * 8);
      *reinterpret_cast<uint4*>(q_s + (ch >> 3) * (FILLTC_Q_ROWS * 128) + r * 128 + (((ch & 7) ^ (r & 7)) << 4)) = w;
    }
  }
  fence_proxy_async_smem();   // the tensor cores read Q through the asynchronous proxy
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  const uint32_t tm_o = 128;                                         // S of tile i at column 64 (i & 1), O at 128

  if (warp == FILLTC_SOFTMAX_THREADS / 32) {
    // ======================= copy + tensor-core issue: one thread =======================
    // K and V have one buffer each.  The tensor cores execute what this thread issues in order:
    //   S(0) | S(1) | O+=PV(0) | S(2) | O+=PV(1) | S(3) | ...
    // S of a tile is issued as soon as its K tile has landed (the S buffer it overwrites was read two tiles ago),
    // so the soft-max threads find their next logits waiting; O += P V of a tile once its weights are written.
    if ((tid & 31) == 0) {
      const uint32_t idesc_s = umma_idesc_bf16(FILLTC_Q_ROWS, KT, false);
      const uint32_t idesc_o = umma_idesc_bf16(FILLTC_Q_ROWS, D, true);
      const uint32_t q_a = smem_addr(q_s), k_a = smem_addr(k_s), v_a = smem_addr(v_s);
      auto load_k = [&](int i) {
        mbar_expect_tx(&bar_k, (uint32_t)T_BYTES);
        const int y = head_row0 + i * KT;
        tma_load_2d_keep(k_s, &map_k, 0, y, &bar_k);
        tma_load_2d_keep(k_s + KT * 128, &map_k, 64, y, &bar_k);
      };
      auto load_v = [&](int i) {
        mbar_expect_tx(&bar_v, (uint32_t)T_BYTES);
        const int y = head_row0 + i * KT;
        tma_load_2d_keep(v_s, &map_v, 0, y, &bar_v);
        tma_load_2d_keep(v_s + KT * 128, &map_v, 64, y, &bar_v);
      };
      // S = Q K^T of tile i into S buffer i & 1: 8 steps of 16 along D; a step moves 32 bytes inside the 128-byte
      // row, 4 steps per box.
      auto issue_qk = [&](int i) {
        tc_fence_after();
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint64_t a = umma_desc_sw128(q_a + (ks >> 2) * (FILLTC_Q_ROWS * 128) + (ks & 3) * 32, 16, 1024);
          const uint64_t bd = umma_desc_sw128(k_a + (ks >> 2) * (KT * 128) + (ks & 3) * 32, 16, 1024);
          umma_bf16(tmem + (uint32_t)(64 * (i & 1)), a, bd, idesc_s, ks > 0 ? 1u : 0u);
        }
        umma_commit(&bar_s[i & 1]);
      };
      load_k(0);
      load_v(0);
      bool okp = fill_wait(&bar_k, 0u);
      if (okp) issue_qk(0);
      if (okp && n_tiles > 1) {
        okp = fill_wait(&bar_s[0], 0u);              // S(0) computed: the K buffer is free
        if (okp) load_k(1);
      }
      for (int i = 0; i < n_tiles && okp; ++i) {
        if (i + 1 < n_tiles) {                       // the next tile's logits, ahead of the soft-max that needs them
          okp = fill_wait(&bar_k, (uint32_t)((i + 1) & 1));
          if (!okp) break;
          issue_qk(i + 1);
        }
        okp = fill_wait(&bar_p, (uint32_t)(i & 1)) && fill_wait(&bar_v, (uint32_t)(i & 1));
        if (!okp) break;
        tc_fence_after();
        // O += P V: 4 steps of 16 state rows; V as stored is MN-major (D contiguous)
        // (the weights sit where the tile's logits were: hi terms in the first 32 columns, lo terms in the other 32)
        const uint32_t tm_p = tmem + (uint32_t)(64 * (i & 1));
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk) {
          const uint64_t bd = umma_desc_sw128(v_a + kk * 2048, KT * 128, 1024);
          umma_bf16_a_tmem(tmem + tm_o, tm_p + kk * 8, bd, idesc_o, (i > 0 || kk > 0) ? 1u : 0u);
          umma_bf16_a_tmem(tmem + tm_o, tm_p + 32 + kk * 8, bd, idesc_o, 1u);
        }
        umma_commit(&bar_o);
        if (i + 2 < n_tiles) {                       // S(i+1) computed: K(i+2) may overwrite K(i+1)
          okp = fill_wait(&bar_s[(i + 1) & 1], (uint32_t)(((i + 1) >> 1) & 1));
          if (!okp) break;
          load_k(i + 2);
        }
        if (i + 1 < n_tiles) {                       // O += P V of tile i completed: V(i+1) may overwrite V(i)
          okp = fill_wait(&bar_o, (uint32_t)(i & 1));
          if (!okp) break;
          load_v(i + 1);
        }
      }
      if (!okp) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    }
  } else {
    // ======================= soft-max: two threads per query row =======================
    // A warp reaches the 32 TMEM lanes of its quarter (warp mod 4); warps 0-3 take the first half of a row's
    // columns, warps 4-7 the second half.  No barrier of the whole CTA inside the loop: the threads meet the
    // issuing thread, and each other, only through the mbarriers.
    const int row = (warp & 3) * 32 + (tid & 31), half = warp >> 2;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int my_t = min(t0 + row, p.F - 1);
    const int vis = p.n0 + my_t;            // last state row this thread's query sees
    float m_run = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int i = 0; i < n_tiles; ++i) {
      const int j0 = i * KT;
      const uint32_t tm_s = (uint32_t)(64 * (i & 1));
      ok = __all_sync(0xffffffffu, fill_wait(&bar_s[i & 1], (uint32_t)((i >> 1) & 1))) != 0;   // this tile's logits
      if (!ok) break;
      tc_fence_after();
      // this thread's half of the row's logits; the two halves exchange their maxima through shared memory
      constexpr int KH = KT / 2;
      float s[KH];
      tmem_ld32(lane_base + tm_s + (uint32_t)(KH * half), s);
      const int jh = j0 + KH * half;
      if (j0 + KT - 1 > p.n0 + t0) {   // some query of this CTA cannot see the whole tile (CTA-uniform)
#pragma unroll
        for (int c = 0; c < KH; ++c) s[c] = (jh + c <= vis) ? s[c] : -INFINITY;
      }
      // (four independent chains: a single running maximum would be 32 dependent instructions)
      float mxa = fmaxf(s[0], s[1]), mxb = fmaxf(s[2], s[3]), mxc = fmaxf(s[4], s[5]), mxd = fmaxf(s[6], s[7]);
#pragma unroll
      for (int c = 8; c < KH; c += 8) {
        mxa = fmaxf(mxa, fmaxf(s[c], s[c + 1]));
        mxb = fmaxf(mxb, fmaxf(s[c + 2], s[c + 3]));
        mxc = fmaxf(mxc, fmaxf(s[c + 4], s[c + 5]));
        mxd = fmaxf(mxd, fmaxf(s[c + 6], s[c + 7]));
      }
      float mx = fmaxf(fmaxf(mxa, mxb), fmaxf(mxc, mxd));
      half_max[i & 1][half][row] = mx;
      // The weights will overwrite the logits' columns: the row's other thread must have read its logits too.
      tc_fence_before();
      named_barrier_sync(1 + (warp & 3), 64);
      tc_fence_after();
      mx = fmaxf(mx, half_max[i & 1][half ^ 1][row]);
      mx *= p.scale2;                             // scale2 > 0: the maximum commutes with the scaling
      const float m_new = fmaxf(m_run, mx);       // finite from tile 0 on: row 0 of the state is visible to every query
      const float corr = exp2_diff(m_run, m_new);
      m_run = m_new;
      // Pairs of logits go through packed fp32 instructions: x = s * scale - m, the row sum, and the lo term
      // e - hi(e) (as hi * -1 + e: one rounding, the same value as the subtraction).
      const uint64_t scale_2 = pack_f2(p.scale2, p.scale2), mneg_2 = pack_f2(-m_new, -m_new);
      const uint64_t minus1_2 = pack_f2(-1.f, -1.f);
      uint64_t lsum2[2] = {pack_f2(0.f, 0.f), pack_f2(0.f, 0.f)};
      uint32_t hi[KH / 2], lo[KH / 2];
#pragma unroll
      for (int e = 0; e < KH / 2; ++e) {
        float x0, x1;
        unpack_f2(fma_f2(pack_f2(s[2 * e], s[2 * e + 1]), scale_2, mneg_2), x0, x1);
        const float e0 = ex2_approx(x0), e1 = ex2_approx(x1);
        const uint64_t e_2 = pack_f2(e0, e1);
        lsum2[e & 1] = add_f2(lsum2[e & 1], e_2);
        const __nv_bfloat162 hb = __floats2bfloat162_rn(e0, e1);
        const uint32_t hw = *reinterpret_cast<const uint32_t*>(&hb);
        float d0, d1;
        unpack_f2(fma_f2(pack_f2(__uint_as_float(hw << 16), __uint_as_float(hw & 0xffff0000u)), minus1_2, e_2), d0, d1);
        const __nv_bfloat162 lb = __floats2bfloat162_rn(d0, d1);
        hi[e] = hw;
        lo[e] = *reinterpret_cast<const uint32_t*>(&lb);
      }
      float ls0, ls1;
      unpack_f2(add_f2(lsum2[0], lsum2[1]), ls0, ls1);
      l_run = l_run * corr + (ls0 + ls1);
      // The weights take the place of the tile's logits in tensor memory, as the A operand of O += P V: the
      // row's 64 hi terms in the first 32 columns of the S buffer (two per column), the lo terms in the other 32.
      // (The buffer of tile i-1, still being read by its contraction, is the other one.)
      tmem_st16(lane_base + tm_s + (uint32_t)(16 * half), hi);
      tmem_st16(lane_base + tm_s + 32u + (uint32_t)(16 * half), lo);
      // Before this thread reports tile i, O += P V of tile i-1 must have completed: O may then be touched, and -
      // since that contraction was only issued once EVERY thread had reported tile i-1 - no thread can report a
      // tile while another still owes the previous one (the barrier counts arrivals, not tiles), nor can the
      // barrier run two phases ahead of the issuing thread.
      if (i > 0) {
        ok = __all_sync(0xffffffffu, fill_wait(&bar_o, (uint32_t)((i - 1) & 1))) != 0;
        if (!ok) break;
        tc_fence_after();
        // O of the tiles so far was accumulated against the old max
        if (__any_sync(0xffffffffu, corr != 1.f)) {
#pragma unroll
          for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
            float o[32];
            tmem_ld32(lane_base + tm_o + c0, o);
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] *= corr;
            tmem_st32(lane_base + tm_o + c0, o);
          }
        }
      }
      tmem_st_wait();
      tc_fence_before();
      mbar_arrive(&bar_p);        // this thread's part of the tile's weights (and of O) is in place
    }
    if (ok && n_tiles > 0) {
      ok = __all_sync(0xffffffffu, fill_wait(&bar_o, (uint32_t)((n_tiles - 1) & 1))) != 0;   // the last O += P V
      tc_fence_after();
    }
    half_sum[half][row] = l_run;
    named_barrier_sync(5, FILLTC_SOFTMAX_THREADS);   // (barriers 1-4 belong to the pairs of warps that share rows)
    if (ok) {
      const float rl = 1.f / (half_sum[0][row] + half_sum[1][row]);
      const int t = t0 + row;
#pragma unroll
      for (int c0 = 64 * half; c0 < 64 * half + 64; c0 += 32) {
        float o[32];
        tmem_ld32(lane_base + tm_o + c0, o);
        if (t < p.F) {
          float4* dst = reinterpret_cast<float4*>(p.out + (((size_t)t * p.B + b) * p.H + h) * D + c0);
#pragma unroll
          for (int c = 0; c < 8; ++c)
            dst[c] = make_float4(o[4 * c] * rl, o[4 * c + 1] * rl, o[4 * c + 2] * rl, o[4 * c + 3] * rl);
        }
      }
    } else if ((tid & 31) == 0) {
      atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(FILLTC_TMEM_COLS) : "memory");
  }
}

}  // namespace tova
