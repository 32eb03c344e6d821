// The two device stages of one TOVA decode step (sm_100a).
//
//   split kernel    : streams the cached K/V rows of one (sequence, KV head,
//                     chunk of rows) through shared memory with bulk
//                     asynchronous copies, computes the logits of the query
//                     heads that share the KV head (Eq. 4), a soft-max partial
//                     (max, sum, weighted V sum) per head and chunk (Eq. 7),
//                     and keeps every logit in an fp32 scratch.
//   combine kernel  : merges the partials into the attention output, forms the
//                     head-averaged weights from the kept logits, takes the
//                     arg-min and overwrites the victim's row with the new
//                     token (Section 4, Eq. 9, Algorithm 1).
//
// Logits are kept in the base-2 domain: s2 = sm_scale * log2(e) * (q . k), so
// weights are exp2(s2 - max2).
#pragma once

#include "tova_device.cuh"

namespace tova {

constexpr int ROWS_PER_WARP = 32;   // cache rows one warp owns in the split kernel
constexpr int MAX_SPLIT_WARPS = 8;  // warps per CTA in the split kernel: 1, 2, 4 or 8
constexpr int COMBINE_THREADS = 128;
constexpr int COMBINE_ROWS = 128;   // candidate rows scored per combine CTA

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
  float2* blockmin;   // [B,nx_max] (lowest mean weight, its candidate index as int bits)
  unsigned* counter;  // [B] tickets of the combine CTAs
  int32_t* status;    // [1]
  int32_t* cur_pos;   // [1] position of the token being processed (set by the split kernel)
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
  int32_t chunk_rows; // rows per split CTA = 32 * warps
  int32_t nx;         // combine CTAs per sequence
  int32_t do_evict;   // n == cap and the policy is on
  float scale2;       // sm_scale * log2(e)
};

// ---------------------------------------------------------------------------
// split kernel
// ---------------------------------------------------------------------------
// grid = (max(n_chunks,1), Hkv, B), block = NW warps.  Warp w of chunk c owns
// rows [c*32*NW + 32*w, +32).  Every lane reads 16 bytes of a row; LPR lanes
// cover a row, so a warp reads RPW = 32/LPR rows per pass and needs LPR passes.
template <typename T, int D, int NW, int GB>
__global__ void __launch_bounds__(NW * 32) tova_split_kernel(const StepParams p) {
  constexpr int EPL = Vec16<T>::N;          // elements per lane
  constexpr int RB = D * (int)sizeof(T);    // bytes per row
  constexpr int LPR = RB / 16;              // lanes per row
  constexpr int RPW = 32 / LPR;             // rows per pass
  constexpr int NP = LPR;                   // passes per warp tile (RPW * NP = 32)
  static_assert(LPR >= 8 && LPR <= 32, "row must be 128..512 bytes");

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* k_tile = smem_raw;                                   // [NW][32][RB]
  unsigned char* v_tile = smem_raw + (size_t)NW * ROWS_PER_WARP * RB; // [NW][32][RB]
  float* w_p = reinterpret_cast<float*>(v_tile + (size_t)NW * ROWS_PER_WARP * RB);  // [NW][GB][32]
  float* w_ml = w_p + NW * GB * 32;                                   // [NW][GB][2]
  float* w_acc = w_ml + NW * GB * 2;                                  // [NW][GB][D]
  __shared__ __align__(8) uint64_t bars[MAX_SPLIT_WARPS][2];

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int lig = lane % LPR;   // lane in row group
  const int sub = lane / LPR;   // which of the RPW rows of a pass
  const int c = blockIdx.x, kvh = blockIdx.y, b = blockIdx.z;
  const int row0 = c * p.chunk_rows + warp * ROWS_PER_WARP;            // first row of this warp
  const int nvalid = min(max(p.n - row0, 0), ROWS_PER_WARP);           // live rows of this warp
  const int my_row = lig * RPW + sub;                                  // row this lane ends up owning

  if (lane == 0 && nvalid > 0) {
    mbar_init(&bars[warp][0], 1);
    mbar_init(&bars[warp][1], 1);
    mbar_fence_init();
  }
  __syncwarp();

  // Everything above touches no global memory; below we read what the previous
  // kernels in the stream wrote.
  pdl_wait();
  pdl_launch_dependents();

  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0)
    *p.cur_pos = (p.pos_t < 0) ? *p.cur_pos + 1 : p.pos_t;

  const size_t kv_row0 = ((size_t)b * p.Hkv + kvh) * p.cap + row0;
  unsigned char* my_k = k_tile + (size_t)warp * ROWS_PER_WARP * RB;
  unsigned char* my_v = v_tile + (size_t)warp * ROWS_PER_WARP * RB;
  if (lane == 0 && nvalid > 0) {
    const uint32_t bytes = (uint32_t)nvalid * RB;
    mbar_expect_tx(&bars[warp][0], bytes);
    bulk_g2s(my_k, static_cast<const unsigned char*>(p.K) + kv_row0 * RB, bytes, &bars[warp][0]);
    mbar_expect_tx(&bars[warp][1], bytes);
    bulk_g2s(my_v, static_cast<const unsigned char*>(p.V) + kv_row0 * RB, bytes, &bars[warp][1]);
  }

  const T* qbase = static_cast<const T*>(p.q) + ((size_t)b * p.H + (size_t)kvh * p.G) * D;

  // The new token (candidate n): its logit per head, done once per (b, kvh)
  // by warp 0 of chunk 0 while the copies are in flight.
  if (c == 0 && warp == 0) {
    const T* kn = static_cast<const T*>(p.k_new) + ((size_t)b * p.Hkv + kvh) * D;
    float kf[EPL];
    Vec16<T>::unpack(*reinterpret_cast<const uint4*>(kn + lig * EPL), kf);
    for (int g = 0; g < p.G; ++g) {
      float qf[EPL];
      Vec16<T>::unpack(*reinterpret_cast<const uint4*>(qbase + (size_t)g * D + lig * EPL), qf);
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(qf[e], kf[e], s);
#pragma unroll
      for (int o = LPR / 2; o >= 1; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      s *= p.scale2;
      if (lane == 0) {
        const size_t bh = (size_t)b * p.H + (size_t)kvh * p.G + g;
        p.logits[bh * p.ld + p.n] = s;
        p.part_ml[bh * p.pc + p.n_chunks] = make_float2(s, 1.f);
      }
    }
  }
  if (c >= p.n_chunks) return;  // empty state: only the new token exists

  bool k_ready = false, v_ready = false, failed = false;

  for (int g0 = 0; g0 < p.G; g0 += GB) {
    // ---- logits of GB heads for this warp's 32 rows -----------------------
    float qf[GB][EPL];
#pragma unroll
    for (int gb = 0; gb < GB; ++gb) {
      const int g = min(g0 + gb, p.G - 1);
      Vec16<T>::unpack(*reinterpret_cast<const uint4*>(qbase + (size_t)g * D + lig * EPL), qf[gb]);
    }
    float s[GB];
    float m[GB], l[GB];
    if (nvalid > 0) {
      if (!k_ready) {
        k_ready = true;
        if (!mbar_wait_bounded(&bars[warp][0], 0)) failed = true;
      }
      float part[GB][NP];
      if (!failed) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          const int r = i * RPW + sub;
          float kf[EPL];
          Vec16<T>::unpack(*reinterpret_cast<const uint4*>(my_k + (size_t)r * RB + lig * 16), kf);
#pragma unroll
          for (int gb = 0; gb < GB; ++gb) {
            float a = 0.f;
#pragma unroll
            for (int e = 0; e < EPL; ++e) a = fmaf(qf[gb][e], kf[e], a);
            part[gb][i] = a;
          }
        }
      } else {
#pragma unroll
        for (int gb = 0; gb < GB; ++gb)
#pragma unroll
          for (int i = 0; i < NP; ++i) part[gb][i] = 0.f;
      }
#pragma unroll
      for (int gb = 0; gb < GB; ++gb) {
        float v = transpose_reduce<NP>(part[gb], lig) * p.scale2;
        // rows past the live range hold stale shared memory: mask them out
        s[gb] = (my_row < nvalid) ? v : -INFINITY;
      }
    } else {
#pragma unroll
      for (int gb = 0; gb < GB; ++gb) s[gb] = -INFINITY;
    }

    // ---- soft-max partial of the warp, weights to shared memory -----------
#pragma unroll
    for (int gb = 0; gb < GB; ++gb) {
      if (g0 + gb < p.G && my_row < nvalid) {
        const size_t bh = (size_t)b * p.H + (size_t)kvh * p.G + g0 + gb;
        p.logits[bh * p.ld + row0 + my_row] = s[gb];
      }
      m[gb] = warp_max(s[gb]);
      const float e = exp2_diff(s[gb], m[gb]);
      l[gb] = warp_sum(e);
      w_p[(warp * GB + gb) * 32 + my_row] = e;
    }
    __syncwarp();

    // ---- weighted V sum ----------------------------------------------------
    float acc[GB][EPL];
#pragma unroll
    for (int gb = 0; gb < GB; ++gb)
#pragma unroll
      for (int e = 0; e < EPL; ++e) acc[gb][e] = 0.f;
    if (nvalid > 0) {
      if (!v_ready) {
        v_ready = true;
        if (!failed && !mbar_wait_bounded(&bars[warp][1], 0)) failed = true;
      }
      if (!failed) {
#pragma unroll
        for (int i = 0; i < NP; ++i) {
          const int r = i * RPW + sub;
          if (r < nvalid) {
            float vf[EPL];
            Vec16<T>::unpack(*reinterpret_cast<const uint4*>(my_v + (size_t)r * RB + lig * 16), vf);
#pragma unroll
            for (int gb = 0; gb < GB; ++gb) {
              const float w = w_p[(warp * GB + gb) * 32 + r];
#pragma unroll
              for (int e = 0; e < EPL; ++e) acc[gb][e] = fmaf(w, vf[e], acc[gb][e]);
            }
          }
        }
      }
    }
    // fold the RPW row groups of the warp together
#pragma unroll
    for (int gb = 0; gb < GB; ++gb)
#pragma unroll
      for (int e = 0; e < EPL; ++e)
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) acc[gb][e] += __shfl_xor_sync(0xffffffffu, acc[gb][e], o);

    // ---- merge the warps of the CTA, write the chunk partial --------------
    if (NW == 1) {
#pragma unroll
      for (int gb = 0; gb < GB; ++gb) {
        if (g0 + gb < p.G && sub == 0) {
          const size_t bh = (size_t)b * p.H + (size_t)kvh * p.G + g0 + gb;
          float* dst = p.part_acc + (bh * (p.pc - 1) + c) * D + lig * EPL;
#pragma unroll
          for (int e = 0; e < EPL; e += 4)
            *reinterpret_cast<float4*>(dst + e) =
                make_float4(acc[gb][e], acc[gb][e + 1], acc[gb][e + 2], acc[gb][e + 3]);
          if (lane == 0) p.part_ml[bh * p.pc + c] = make_float2(m[gb], l[gb]);
        }
      }
    } else {
      if (sub == 0) {
#pragma unroll
        for (int gb = 0; gb < GB; ++gb) {
          float* dst = w_acc + (size_t)(warp * GB + gb) * D + lig * EPL;
#pragma unroll
          for (int e = 0; e < EPL; ++e) dst[e] = acc[gb][e];
          if (lane == 0) {
            w_ml[(warp * GB + gb) * 2 + 0] = m[gb];
            w_ml[(warp * GB + gb) * 2 + 1] = l[gb];
          }
        }
      }
      __syncthreads();
      for (int idx = threadIdx.x; idx < GB * D; idx += NW * 32) {
        const int gb = idx / D, d = idx % D;
        if (g0 + gb < p.G) {
          float M = -INFINITY;
#pragma unroll
          for (int w = 0; w < NW; ++w) M = fmaxf(M, w_ml[(w * GB + gb) * 2]);
          float a = 0.f, L = 0.f;
#pragma unroll
          for (int w = 0; w < NW; ++w) {
            const float f = exp2_diff(w_ml[(w * GB + gb) * 2], M);
            a = fmaf(w_acc[(size_t)(w * GB + gb) * D + d], f, a);
            L = fmaf(w_ml[(w * GB + gb) * 2 + 1], f, L);
          }
          const size_t bh = (size_t)b * p.H + (size_t)kvh * p.G + g0 + gb;
          p.part_acc[(bh * (p.pc - 1) + c) * D + d] = a;
          if (d == 0) p.part_ml[bh * p.pc + c] = make_float2(M, L);
        }
      }
      __syncthreads();
    }
  }
  if (failed && lane == 0) atomicExch(p.status, DEV_ERR_COPY_TIMEOUT);
}


// ---------------------------------------------------------------------------
// combine-and-evict kernel
// ---------------------------------------------------------------------------
// grid = (nx, B), block = COMBINE_THREADS.  Every CTA of a sequence first
// rebuilds each head's global (max2, 1/sum) from the chunk partials; CTA x then
//   - writes the attention output of heads x, x+nx, ... (Eq. 7),
//   - scores candidates [x*COMBINE_ROWS, +COMBINE_ROWS): the mean over heads of
//     the soft-max weights (Algorithm 1), and leaves its lowest (value, index).
// The last CTA of the sequence to finish (atomic ticket, no waiting) picks the
// overall arg-min - lowest index on ties - and replaces that row by the new
// token in K, V and the position table (Eq. 9, in place).
// smem: float hM[H], hInvL[H], wts[pc].
template <typename T, int D>
__global__ void __launch_bounds__(COMBINE_THREADS) tova_combine_kernel(const StepParams p) {
  extern __shared__ __align__(16) float csm[];
  float* hM = csm;              // [H]
  float* hInvL = csm + p.H;     // [H]
  float* wts = csm + 2 * p.H;   // [pc]
  __shared__ float red_v[COMBINE_THREADS / 32];
  __shared__ int red_i[COMBINE_THREADS / 32];
  __shared__ int s_last;

  const int x = blockIdx.x, b = blockIdx.y;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int np = p.n_chunks + 1;  // partials per head: the chunks, then the new token

  pdl_wait();
  pdl_launch_dependents();
  const int pos_t = *p.cur_pos;

  // ---- global max and sum of every head ------------------------------------
  for (int h = warp; h < p.H; h += COMBINE_THREADS / 32) {
    const float2* ml = p.part_ml + ((size_t)b * p.H + h) * p.pc;
    float M = -INFINITY;
    for (int i = lane; i < np; i += 32) M = fmaxf(M, ml[i].x);
    M = warp_max(M);
    float L = 0.f;
    for (int i = lane; i < np; i += 32) {
      const float2 e = ml[i];
      L = fmaf(e.y, exp2_diff(e.x, M), L);
    }
    L = warp_sum(L);
    if (lane == 0) {
      hM[h] = M;
      hInvL[h] = 1.f / L;
    }
  }
  __syncthreads();

  // ---- attention output of this CTA's heads --------------------------------
  for (int h = x; h < p.H; h += p.nx) {
    const size_t bh = (size_t)b * p.H + h;
    const float2* ml = p.part_ml + bh * p.pc;
    for (int i = tid; i < np; i += COMBINE_THREADS) wts[i] = exp2_diff(ml[i].x, hM[h]) * hInvL[h];
    __syncthreads();
    const float* acc = p.part_acc + bh * (size_t)(p.pc - 1) * D;
    const T* vn = static_cast<const T*>(p.v_new) + ((size_t)b * p.Hkv + h / p.G) * D;
    for (int d = tid; d < D; d += COMBINE_THREADS) {
      float o = 0.f;
      for (int i = 0; i < p.n_chunks; ++i) o = fmaf(acc[(size_t)i * D + d], wts[i], o);
      o = fmaf((float)vn[d], wts[p.n_chunks], o);
      p.out[bh * D + d] = o;
    }
    __syncthreads();
  }

  constexpr int RB16 = D * (int)sizeof(T) / 16;  // 16-byte words per row
  const int row_words = p.Hkv * RB16;

  if (!p.do_evict) {
    // g(t) = min(t, k) not yet reached: the new token takes the next free row.
    if (x == 0) {
      for (int i = tid; i < row_words; i += COMBINE_THREADS) {
        const int kvh = i / RB16, wd = i % RB16;
        const size_t dst = (((size_t)b * p.Hkv + kvh) * p.cap + p.n) * RB16 + wd;
        const size_t src = ((size_t)b * p.Hkv + kvh) * RB16 + wd;
        static_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[src];
        static_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[src];
      }
      if (tid == 0) {
        p.pos[(size_t)b * p.cap + p.n] = pos_t;
        p.len[b] = p.n + 1;
        if (p.evicted) p.evicted[b] = -1;
      }
    }
    return;
  }

  // ---- head-averaged weight of this CTA's candidates ------------------------
  const int j = x * COMBINE_ROWS + tid;
  float val = INFINITY;
  if (j <= p.n) {
    const float* lg = p.logits + (size_t)b * p.H * p.ld + j;
    float a = 0.f;
    for (int h = 0; h < p.H; ++h) a += exp2f(lg[(size_t)h * p.ld] - hM[h]) * hInvL[h];
    val = a * (1.f / (float)p.H);
  }
  int idx = j;
  // lowest (value, index) of the block
#pragma unroll
  for (int o = 16; o >= 1; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, val, o);
    const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
    if (ov < val || (ov == val && oi < idx)) { val = ov; idx = oi; }
  }
  if (lane == 0) { red_v[warp] = val; red_i[warp] = idx; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < COMBINE_THREADS / 32; ++w)
      if (red_v[w] < val || (red_v[w] == val && red_i[w] < idx)) { val = red_v[w]; idx = red_i[w]; }
    p.blockmin[(size_t)b * p.nx + x] = make_float2(val, __int_as_float(idx));
    __threadfence();
    const unsigned t = atomicAdd(p.counter + b, 1u);
    s_last = (t == (unsigned)p.nx - 1u);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- last CTA of the sequence: arg-min over blocks, evict, insert --------
  if (tid == 0) {
    const volatile float2* bm = p.blockmin + (size_t)b * p.nx;
    float bv = INFINITY;
    int bi = p.n;  // a valid default; every block reports a finite value in practice
    for (int i = 0; i < p.nx; ++i) {
      const float v = bm[i].x;
      const int ci = __float_as_int(bm[i].y);
      if (v < bv || (v == bv && ci < bi)) { bv = v; bi = ci; }
    }
    if (bi < 0 || bi > p.cap) { atomicExch(p.status, DEV_ERR_BAD_VICTIM); bi = p.cap; }
    red_i[0] = bi;
    p.counter[b] = 0;  // ready for the next step
  }
  __syncthreads();
  const int victim = red_i[0];
  if (victim < p.cap) {
    for (int i = tid; i < row_words; i += COMBINE_THREADS) {
      const int kvh = i / RB16, wd = i % RB16;
      const size_t dst = (((size_t)b * p.Hkv + kvh) * p.cap + victim) * RB16 + wd;
      const size_t src = ((size_t)b * p.Hkv + kvh) * RB16 + wd;
      static_cast<uint4*>(p.K)[dst] = static_cast<const uint4*>(p.k_new)[src];
      static_cast<uint4*>(p.V)[dst] = static_cast<const uint4*>(p.v_new)[src];
    }
  }
  if (tid == 0) {
    int ev = pos_t;  // the new token dropped itself
    if (victim < p.cap) {
      ev = p.pos[(size_t)b * p.cap + victim];
      p.pos[(size_t)b * p.cap + victim] = pos_t;
    }
    if (p.evicted) p.evicted[b] = ev;
  }
}

// Empty state at init: length 0, positions -1, counters and status 0.
__global__ void tova_init_kernel(int32_t* pos, int32_t* len, unsigned* counter, int32_t* status,
                                 int32_t* cur_pos, int B, int cap) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < (size_t)B * cap) pos[i] = -1;
  if (i < (size_t)B) { len[i] = 0; counter[i] = 0; }
  if (i == 0) { *status = 0; *cur_pos = -1; }
}

}  // namespace tova
