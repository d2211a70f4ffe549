// Row-wise pair-biased attention core for bf16, head dims 16 / 32 / 64.
//
// One CTA owns 128 queries j of one (sample, head) and walks a chunk of attention rows i (pair
// order) or the single row of a sample (token order).  The bias tile bias[h][j0:j0+128][:] is the
// same for every row i of the sample, so it is fetched once per CTA and stays in shared memory
// (samples too long for that read it through L1/L2 instead).  A producer warp streams the rows' Q
// tile and 64-key K / V blocks with TMA (swizzled so ldmatrix is conflict-free) through mbarrier
// rings; eight consumer warps (16 queries each) compute scores and P.V on the tensor cores
// (m16n8k16 bf16, P kept in registers between the two products) with the online softmax
// (running max / running sum) in float, in the log2 domain.
// The core is bound by the softmax arithmetic, not by the tensor pipe: per score element there
// are 2 d tensor flops against ~7 CUDA-core instructions and one exponential.
#include <cstring>

#include "fast.cuh"
#include "tc_common.cuh"

namespace ntp {

constexpr int AT_Q = 128;         // queries per CTA
constexpr int AT_K = 64;          // keys per pipeline step
constexpr int AT_STAGES = 4;
constexpr int AT_CONSUMERS = 8;
constexpr int AT_THREADS = 32 + AT_CONSUMERS * 32;
constexpr int AT_RES_CAP = 100 * 1024;   // largest resident bias tile (bytes)
constexpr float LOG2E = 1.4426950408889634f;

struct AttnCoreParams {
  CUtensorMap qmap, kmap, vmap;   // flat {H d, rows}; boxes {d, 128} (q) and {d, 64} (k, v)
  BatchMeta m;
  const __nv_bfloat16* bias;      // head-major channel-major, nullable
  __nv_bfloat16* o;
  long long row0;                 // first row the maps cover
  int H, pair_order, ichunk, bias_bytes;
  float bias_mul;                 // factor that brings the stored bias to bias * sqrt(d) (1 if stored that way)
  int bias_prescaled;             // bias buffer already holds bias * sqrt(d): the resident tile can go through the MMA
  int skip_max_n;                 // samples with N <= skip_max_n belong to the tcgen05 kernel
  int* status;
};

__host__ __device__ inline int at_bias_stride(int N) {   // bytes per resident bias row: 16 mod 32
  int b = round_up8(N) * 2;
  return (b / 16) % 2 == 0 ? b + 16 : b;
}

__device__ inline void cp_async16(void* smem, const void* gmem, bool valid) {
  const unsigned sa = (unsigned)__cvta_generic_to_shared(smem);
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(sa), "l"(gmem), "r"(sz));
}
__device__ inline void cp_async_wait_all() { asm volatile("cp.async.wait_all;\n" ::: "memory"); }

__device__ inline void ldsm_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, unsigned a) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ inline void ldsm_x2(unsigned& r0, unsigned& r1, unsigned a) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r0), "=r"(r1) : "r"(a));
}
__device__ inline void ldsm_x4_t(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, unsigned a) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ inline void mma_bf16(float (&c)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline unsigned pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<unsigned*>(&h);
}
// two exponentials at once: the arguments are rounded to bf16 (they are <= 0, so the absolute error grows
// only where the weight is already small) and the results come back packed as the bf16 pair the PV MMA takes
__device__ inline unsigned exp2_bf16x2(float lo, float hi) {
  unsigned x, y;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;\n" : "=r"(x) : "f"(hi), "f"(lo));
  asm("ex2.approx.ftz.bf16x2 %0, %1;\n" : "=r"(y) : "r"(x));
  return y;
}
__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

// byte offset of 16-byte chunk `chunk` of row `row` in a TMA tile with rows of 2 D bytes and the
// swizzle span equal to the row (32 / 64 / 128 bytes): chunk bits are XORed with address bits [7, ..)
template <int D>
__device__ inline unsigned tile_off(int row, int chunk) {
  constexpr int ROWB = 2 * D, CH = ROWB / 16;
  return row * ROWB + (((chunk ^ ((row * ROWB) >> 7)) & (CH - 1)) << 4);
}

__device__ inline void mma_bf16_zero(float (&d)[4], const unsigned (&a)[4], unsigned b0, unsigned b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};\n"
               : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.0f));
}

// One 64-key (NT = 8) or 32-key (NT = 4) step of 16 queries.
// BIAS: 0 none; 1 resident tile stored pre-multiplied by sqrt(d), added on the tensor cores by an
// extra MMA whose A operand is the 16 x 16 identity (1.0 * bias is exact in the float accumulator);
// 2 read through L1/L2 and multiplied by bias_mul on the CUDA cores.
// Scores stay in unscaled units S' = q.k + bias sqrt(d); the softmax scale log2(e) / sqrt(d) is
// applied inside the exponent: p = exp2(sc2 S' - sc2 max').
template <int D, int NT, int BIAS, bool MASKED>
__device__ inline void attn_step(float (&sacc)[AT_K / 8][4], float (&oacc)[D / 8][4], float (&mrow)[2], float (&lacc)[4],
                                 const unsigned (&qf)[D / 16][4], const unsigned (&idf)[4], unsigned ks_, unsigned vs_,
                                 unsigned bias_s, int ld, const __nv_bfloat16* bg0, const __nv_bfloat16* bg1, int k0,
                                 int N, float sc2, float bias_mul, int lane) {
  const int tq = lane & 3;
  // ---- S' = bias' + Q K^T for 16 queries x (8 NT) keys
#pragma unroll
  for (int nt = 0; nt < NT; nt += 2) {
    if constexpr (BIAS == 1) {
      // bias^T fragments of key tiles nt and nt + 1: (query rows 0-7 | 8-15) x (8 keys), transposed on load
      unsigned b0 = 0, b1 = 0, b2 = 0, b3 = 0;
      if (!MASKED || k0 + nt * 8 < ld) ldsm_x4_t(b0, b1, b2, b3, bias_s + ((lane >> 4) + nt) * 16);
      mma_bf16_zero(sacc[nt], idf, b0, b1);
      mma_bf16_zero(sacc[nt + 1], idf, b2, b3);
    }
  }
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int krow = nt * 8 + (lane & 7);
    if constexpr (D == 16) {
      unsigned b0, b1;
      ldsm_x2(b0, b1, ks_ + tile_off<D>(krow, (lane >> 3) & 1));
      if constexpr (BIAS == 1) mma_bf16(sacc[nt], qf[0], b0, b1);
      else mma_bf16_zero(sacc[nt], qf[0], b0, b1);
    } else {
#pragma unroll
      for (int kp = 0; kp < D / 32; ++kp) {
        unsigned b0, b1, b2, b3;
        ldsm_x4(b0, b1, b2, b3, ks_ + tile_off<D>(krow, kp * 4 + (lane >> 3)));
        if (BIAS == 1 || kp > 0) mma_bf16(sacc[nt], qf[kp * 2], b0, b1);
        else mma_bf16_zero(sacc[nt], qf[kp * 2], b0, b1);
        mma_bf16(sacc[nt], qf[kp * 2 + 1], b2, b3);
      }
    }
  }
  // ---- bias through L1/L2 (long samples), mask, running max
  float t0[2] = {-INFINITY, -INFINITY}, t1[2] = {-INFINITY, -INFINITY};   // two chains each, half the latency
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int kc = k0 + nt * 8 + 2 * tq;
    if constexpr (BIAS == 2) {
      unsigned w0 = 0, w1 = 0;
      if (!MASKED || kc < ld) {
        w0 = __ldg(reinterpret_cast<const unsigned*>(bg0 + kc));
        w1 = __ldg(reinterpret_cast<const unsigned*>(bg1 + kc));
      }
      sacc[nt][0] = fmaf(__uint_as_float(w0 << 16), bias_mul, sacc[nt][0]);
      sacc[nt][1] = fmaf(__uint_as_float(w0 & 0xffff0000u), bias_mul, sacc[nt][1]);
      sacc[nt][2] = fmaf(__uint_as_float(w1 << 16), bias_mul, sacc[nt][2]);
      sacc[nt][3] = fmaf(__uint_as_float(w1 & 0xffff0000u), bias_mul, sacc[nt][3]);
    }
    if constexpr (MASKED) {
      if (kc >= N) sacc[nt][0] = sacc[nt][2] = -INFINITY;
      if (kc + 1 >= N) sacc[nt][1] = sacc[nt][3] = -INFINITY;
    }
    t0[nt & 1] = fmaxf(t0[nt & 1], fmaxf(sacc[nt][0], sacc[nt][1]));
    t1[nt & 1] = fmaxf(t1[nt & 1], fmaxf(sacc[nt][2], sacc[nt][3]));
  }
  float mx0 = fmaxf(t0[0], t0[1]), mx1 = fmaxf(t1[0], t1[1]);
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  const float mn0 = fmaxf(mrow[0], mx0), mn1 = fmaxf(mrow[1], mx1);   // finite: key k0 is valid
  const float cr0 = fast_exp2((mrow[0] - mn0) * sc2), cr1 = fast_exp2((mrow[1] - mn1) * sc2);
  mrow[0] = mn0;
  mrow[1] = mn1;
  const float ms0 = -mn0 * sc2, ms1 = -mn1 * sc2;
#pragma unroll
  for (int nd = 0; nd < D / 8; ++nd) {
    oacc[nd][0] *= cr0; oacc[nd][1] *= cr0;
    oacc[nd][2] *= cr1; oacc[nd][3] *= cr1;
  }
  lacc[0] *= cr0; lacc[1] *= cr0;
  lacc[2] *= cr1; lacc[3] *= cr1;
  // ---- O += P V, with the row sums of P accumulated by one more MMA against an all-ones B tile, so the
  // denominator sums exactly the rounded weights the numerator uses
#pragma unroll
  for (int kk = 0; kk < NT / 2; ++kk) {
    unsigned pf[4];
    pf[0] = exp2_bf16x2(fmaf(sacc[2 * kk][0], sc2, ms0), fmaf(sacc[2 * kk][1], sc2, ms0));
    pf[1] = exp2_bf16x2(fmaf(sacc[2 * kk][2], sc2, ms1), fmaf(sacc[2 * kk][3], sc2, ms1));
    pf[2] = exp2_bf16x2(fmaf(sacc[2 * kk + 1][0], sc2, ms0), fmaf(sacc[2 * kk + 1][1], sc2, ms0));
    pf[3] = exp2_bf16x2(fmaf(sacc[2 * kk + 1][2], sc2, ms1), fmaf(sacc[2 * kk + 1][3], sc2, ms1));
    mma_bf16(lacc, pf, 0x3F803F80u, 0x3F803F80u);
#pragma unroll
    for (int np = 0; np < D / 16; ++np) {
      const int mtx = lane >> 3;
      const int krow = kk * 16 + (mtx & 1) * 8 + (lane & 7);
      unsigned b0, b1, b2, b3;
      ldsm_x4_t(b0, b1, b2, b3, vs_ + tile_off<D>(krow, np * 2 + (mtx >> 1)));
      mma_bf16(oacc[np * 2], pf, b0, b1);
      mma_bf16(oacc[np * 2 + 1], pf, b2, b3);
    }
  }
}

template <int D, int BIAS>
__device__ inline void attn_step_dispatch(bool masked, int rem, float (&sacc)[AT_K / 8][4], float (&oacc)[D / 8][4],
                                          float (&mrow)[2], float (&lacc)[4], const unsigned (&qf)[D / 16][4],
                                          const unsigned (&idf)[4], unsigned ks_, unsigned vs_, unsigned bias_s, int ld,
                                          const __nv_bfloat16* bg0, const __nv_bfloat16* bg1, int k0, int N, float sc2,
                                          float bias_mul, int lane) {
  if (!masked)
    attn_step<D, 8, BIAS, false>(sacc, oacc, mrow, lacc, qf, idf, ks_, vs_, bias_s, ld, bg0, bg1, k0, N, sc2, bias_mul, lane);
  else if (rem > 32)
    attn_step<D, 8, BIAS, true>(sacc, oacc, mrow, lacc, qf, idf, ks_, vs_, bias_s, ld, bg0, bg1, k0, N, sc2, bias_mul, lane);
  else
    attn_step<D, 4, BIAS, true>(sacc, oacc, mrow, lacc, qf, idf, ks_, vs_, bias_s, ld, bg0, bg1, k0, N, sc2, bias_mul, lane);
}

// BIAS: 0 = no bias, 1 = bias tile resident in shared memory (samples with want_resident), 2 = bias through L1/L2.
// A launch handles the samples whose bias tile fits (BIAS == 1) or the ones whose tile does not (BIAS == 2).
template <int D, int BIAS>
__global__ void __launch_bounds__(AT_THREADS, 2) attn_core_kernel(const __grid_constant__ AttnCoreParams p) {
  constexpr int KV_TILE = AT_K * D * 2;      // bytes of one K or V block
  constexpr int Q_TILE = AT_Q * D * 2;
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * AT_STAGES + 4];
  __shared__ int s_item[4];
  __shared__ int abort_flag;
  unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
  unsigned char* sK = smem;                               // [STAGES][64][2D]
  unsigned char* sV = sK + AT_STAGES * KV_TILE;
  unsigned char* sQ = sV + AT_STAGES * KV_TILE;           // [2][128][2D]
  unsigned char* sB = sQ + 2 * Q_TILE;                    // resident bias tile [128][bstride]
  unsigned long long* kvfull = bars;
  unsigned long long* kvempty = bars + AT_STAGES;
  unsigned long long* qfull = bars + 2 * AT_STAGES;
  unsigned long long* qempty = bars + 2 * AT_STAGES + 2;
  const BatchMeta& m = p.m;
  const int H = p.H, pair_order = p.pair_order;

  if (threadIdx.x == 0) {
    long long w = blockIdx.x;
    int s = 0;
    for (; s < m.B; ++s) {
      const int N = m.N[s];
      if (N <= p.skip_max_n) continue;
      if (BIAS != 0 && (AT_Q * at_bias_stride(N) <= AT_RES_CAP) != (BIAS == 1)) continue;   // other launch's sample
      const long long njb = (N + AT_Q - 1) / AT_Q;
      const long long nic = pair_order ? (N + p.ichunk - 1) / p.ichunk : (N > 0 ? 1 : 0);
      const long long cnt = njb * H * nic;
      if (w < cnt) break;
      w -= cnt;
    }
    s_item[0] = s;
    if (s < m.B) {
      const int N = m.N[s];
      const int njb = (N + AT_Q - 1) / AT_Q;
      s_item[1] = (int)(w % njb);                  // j block
      s_item[2] = (int)((w / njb) % H);            // head
      s_item[3] = (int)(w / ((long long)njb * H)); // i chunk
    }
    abort_flag = 0;
  }
  __syncthreads();
  const int s = s_item[0];
  if (s >= m.B) return;
  const int N = m.N[s], ld = round_up8(N);
  const int j0 = s_item[1] * AT_Q, h = s_item[2];
  const int i_begin = pair_order ? s_item[3] * p.ichunk : 0;
  const int i_end = pair_order ? min(N, i_begin + p.ichunk) : 1;
  const int Hd = H * D;
  const int nkb = (N + AT_K - 1) / AT_K;
  const int n_active = min(AT_CONSUMERS, (N - j0 + 15) / 16);   // consumer warps that own valid queries
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  constexpr bool has_bias = BIAS != 0;
  const int bstride = at_bias_stride(N);
  constexpr bool resident = BIAS == 1;
  const __nv_bfloat16* bias_h =
      has_bias ? p.bias + (long long)H * m.cm_off[s] + (long long)h * N * ld : nullptr;
  if (threadIdx.x == 0) {
    for (int st = 0; st < AT_STAGES; ++st) { mbar_init(&kvfull[st], 1); mbar_init(&kvempty[st], n_active); }
    for (int st = 0; st < 2; ++st) { mbar_init(&qfull[st], 1); mbar_init(&qempty[st], n_active); }
    mbar_fence_init();
  }
  // ---- resident bias tile: rows j0..j0+127, all keys (loaded by the consumer threads)
  if (resident && warp > 0) {
    const int chunks = ld / 8;
    for (int idx = threadIdx.x - 32; idx < AT_Q * chunks; idx += AT_CONSUMERS * 32) {
      const int r = idx / chunks, c = idx - r * chunks;
      const bool ok = j0 + r < N;
      cp_async16(sB + r * bstride + c * 16, bias_h + (long long)(ok ? j0 + r : 0) * ld + c * 8, ok);
    }
    cp_async_wait_all();
  }
  __syncthreads();
  AbortCtx ab{p.status, &abort_flag};
  auto row_coord = [&](int i) -> long long {   // first packed row of attention row i, relative to the maps
    return (pair_order ? m.pair_off[s] + (long long)i * N : m.tok_off[s]) - p.row0;
  };

  if (warp == 0) {
    if (lane != 0) return;
    // ------------------------------------------------------------------ TMA producer
    int st = 0, qs = 0;
    unsigned ph = 0, qph = 0;
    for (int i = i_begin; i < i_end; ++i) {
      const int base = (int)row_coord(i);
      mbar_wait(&qempty[qs], qph ^ 1, ab);
      mbar_expect_tx(&qfull[qs], Q_TILE);
      tma_load_2d(sQ + qs * Q_TILE, &p.qmap, &qfull[qs], h * D, base + j0);
      if (++qs == 2) { qs = 0; qph ^= 1; }
      for (int kb = 0; kb < nkb; ++kb) {
        mbar_wait(&kvempty[st], ph ^ 1, ab);
        mbar_expect_tx(&kvfull[st], 2 * KV_TILE);
        tma_load_2d(sK + st * KV_TILE, &p.kmap, &kvfull[st], h * D, base + kb * AT_K);
        tma_load_2d(sV + st * KV_TILE, &p.vmap, &kvfull[st], h * D, base + kb * AT_K);
        if (++st == AT_STAGES) { st = 0; ph ^= 1; }
      }
    }
    return;
  }
  // -------------------------------------------------------------------- consumers
  const int cw = warp - 1;
  if (cw >= n_active) return;
  const int g = lane >> 2, tq = lane & 3;
  const float sc2 = rsqrtf((float)D) * LOG2E;
  const bool tail = (N % AT_K) != 0;
  unsigned qf[D / 16][4];
  float oacc[D / 8][4];
  float sacc[AT_K / 8][4];
  float mrow[2], lacc[4];
  const int rloc = cw * 16 + g;                       // this thread's first query row inside the CTA tile
  // identity A fragment of the bias MMA: 1.0 where the query row equals the k index
  unsigned idf[4];
  idf[0] = idf[3] = (g == 2 * tq ? 0x00003F80u : 0u) | (g == 2 * tq + 1 ? 0x3F800000u : 0u);
  idf[1] = idf[2] = 0u;
  // ldmatrix lane address into the resident bias tile: query row ((lane >> 3) & 1) * 8 + (lane & 7) of this warp
  const unsigned bias_lane = smem_u32(sB) + (cw * 16 + ((lane >> 3) & 1) * 8 + (lane & 7)) * bstride;
  const int jr0 = min(j0 + rloc, N - 1), jr1 = min(j0 + rloc + 8, N - 1);
  const __nv_bfloat16* bg0 = has_bias ? bias_h + (long long)jr0 * ld : nullptr;
  const __nv_bfloat16* bg1 = has_bias ? bias_h + (long long)jr1 * ld : nullptr;
  int st = 0, qs = 0;
  unsigned ph = 0, qph = 0;
  for (int i = i_begin; i < i_end; ++i) {
    mbar_wait(&qfull[qs], qph, ab);
    {
      const unsigned qbase = smem_u32(sQ + qs * Q_TILE);
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int mtx = lane >> 3;
        const int row = cw * 16 + (mtx & 1) * 8 + (lane & 7);
        ldsm_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], qbase + tile_off<D>(row, ks * 2 + (mtx >> 1)));
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&qempty[qs]);
    if (++qs == 2) { qs = 0; qph ^= 1; }
#pragma unroll
    for (int nd = 0; nd < D / 8; ++nd) oacc[nd][0] = oacc[nd][1] = oacc[nd][2] = oacc[nd][3] = 0.f;
    mrow[0] = mrow[1] = -INFINITY;
    lacc[0] = lacc[1] = lacc[2] = lacc[3] = 0.f;
    for (int kb = 0; kb < nkb; ++kb) {
      mbar_wait(&kvfull[st], ph, ab);
      const unsigned ks_ = smem_u32(sK + st * KV_TILE), vs_ = smem_u32(sV + st * KV_TILE);
      const int k0 = kb * AT_K;
      const bool masked = tail && kb == nkb - 1;
      const unsigned bias_s = bias_lane + k0 * 2;
      attn_step_dispatch<D, BIAS>(masked, N - k0, sacc, oacc, mrow, lacc, qf, idf, ks_, vs_, bias_s, ld, bg0, bg1, k0, N,
                                  sc2, p.bias_mul, lane);
      __syncwarp();
      if (lane == 0) mbar_arrive(&kvempty[st]);
      if (++st == AT_STAGES) { st = 0; ph ^= 1; }
    }
    // ---- normalise and store this row's 16 x d outputs
    const float inv0 = 1.0f / lacc[0], inv1 = 1.0f / lacc[2];   // every column of the ones tile holds the row sum
    const long long base = row_coord(i) + p.row0;
    const int r0 = j0 + rloc, r1 = r0 + 8;
#pragma unroll
    for (int nd = 0; nd < D / 8; ++nd) {
      const int col = h * D + nd * 8 + 2 * tq;
      if (r0 < N)
        *reinterpret_cast<unsigned*>(p.o + (base + r0) * Hd + col) = pack_bf16(oacc[nd][0] * inv0, oacc[nd][1] * inv0);
      if (r1 < N)
        *reinterpret_cast<unsigned*>(p.o + (base + r1) * Hd + col) = pack_bf16(oacc[nd][2] * inv1, oacc[nd][3] * inv1);
    }
  }
}

bool fast_attn_core_supported(int H, int d) { return (d == 16 || d == 32 || d == 64) && H >= 1; }

template <int D, int BIAS>
static nt_status launch_attn_mode(AttnCoreParams& p, int bias_bytes, cudaStream_t st) {
  const BatchMeta& m = p.m;
  auto count = [&](int ic) {
    long long c = 0;
    for (int s = 0; s < m.B; ++s) {
      const long long N = m.N[s], njb = (N + AT_Q - 1) / AT_Q;
      if (N <= p.skip_max_n) continue;
      if (BIAS != 0 && (AT_Q * at_bias_stride((int)N) <= AT_RES_CAP) != (BIAS == 1)) continue;
      const long long nic = p.pair_order ? (N + ic - 1) / ic : (N > 0 ? 1 : 0);
      c += njb * p.H * nic;
    }
    return c;
  };
  int ichunk = 32;
  while (p.pair_order && ichunk > 2 && count(ichunk) < 148 * 12) ichunk >>= 1;
  p.ichunk = ichunk;
  const long long blocks = count(ichunk);
  if (blocks == 0) return NT_OK;
  if (blocks > 0x7FFFFFFFll) return NT_ERR_UNSUPPORTED;
  const size_t smem = (size_t)2 * AT_STAGES * AT_K * D * 2 + 2 * (size_t)AT_Q * D * 2 + (BIAS == 1 ? bias_bytes + 128 : 0) + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_core_kernel<D, BIAS>, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024) !=
        cudaSuccess)
      return cuda_fail("attention core smem attribute");
    attr_set = true;
  }
  {
    LaunchScope ls("attn_core", st);
    attn_core_kernel<D, BIAS><<<(unsigned)blocks, AT_THREADS, smem, st>>>(p);
  }
  return cuda_ok("attention core launch");
}

template <int D>
static nt_status launch_attn(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                             const __nv_bfloat16* bias, __nv_bfloat16* o, int H, int pair_order, int bias_prescaled,
                             const BatchMeta& m, int* status, cudaStream_t st) {
  AttnCoreParams p;
  memset(&p, 0, sizeof(p));
  p.m = m;
  p.bias = bias;
  p.o = o;
  p.H = H;
  p.pair_order = pair_order;
  p.bias_prescaled = bias_prescaled;
  p.bias_mul = bias_prescaled ? 1.0f : sqrtf((float)D);
  p.status = status;
  // a bias must come stored times sqrt(d) (as the tensor-core input projection writes it)
  if (bias && !bias_prescaled) return NT_ERR_UNSUPPORTED;
  p.row0 = pair_order ? m.pair_off[0] : m.tok_off[0];
  const long long rows = (pair_order ? m.pair_off[m.B] : m.tok_off[m.B]) - p.row0;
  if (rows <= 0) return NT_OK;
  if (rows > 0x7FFFFF00ll) return NT_ERR_UNSUPPORTED;
  // short samples (pair order) go to the tcgen05 kernel, which holds a whole score row in TMEM
  int skip = 0;
  if (pair_order && (D == 16 || D == 32)) {
    const int n_tc = fast_attn_tc_max_n(D, bias != nullptr);
    bool any_short = false, any_other = false;
    for (int s = 0; s < m.B; ++s) {
      if (m.N[s] >= 1 && m.N[s] <= n_tc) any_short = true;
      else if (m.N[s] > n_tc) any_other = true;
    }
    if (any_short) {
      const nt_status r = fast_attn_core_tc(q, k, v, bias, o, H, D, m, n_tc, status, st);
      if (r != NT_OK) return r;
      skip = n_tc;
      if (!any_other) return NT_OK;
    }
  }
  p.skip_max_n = skip;
  int bias_bytes = 0;
  bool any_long = false;
  for (int s = 0; s < m.B; ++s) {
    if (m.N[s] <= skip) continue;
    const int res = AT_Q * at_bias_stride(m.N[s]);
    if (res <= AT_RES_CAP) { if (res > bias_bytes) bias_bytes = res; }
    else any_long = true;
  }
  p.bias_bytes = bias_bytes;
  const int Hd = H * D;
  {
    const unsigned long long dims[2] = {(unsigned long long)Hd, (unsigned long long)rows};
    const unsigned long long strides[1] = {(unsigned long long)Hd * 2};
    const unsigned qbox[2] = {(unsigned)D, AT_Q}, kbox[2] = {(unsigned)D, AT_K};
    if (!make_tmap_16bit(&p.qmap, q + p.row0 * Hd, 2, dims, strides, qbox, 2 * D)) return cuda_fail("attn q map");
    if (!make_tmap_16bit(&p.kmap, k + p.row0 * Hd, 2, dims, strides, kbox, 2 * D)) return cuda_fail("attn k map");
    if (!make_tmap_16bit(&p.vmap, v + p.row0 * Hd, 2, dims, strides, kbox, 2 * D)) return cuda_fail("attn v map");
  }
  if (!bias) return launch_attn_mode<D, 0>(p, 0, st);
  nt_status r = launch_attn_mode<D, 1>(p, bias_bytes, st);
  if (r != NT_OK) return r;
  if (any_long) r = launch_attn_mode<D, 2>(p, 0, st);
  return r;
}

nt_status fast_attn_core(const void* q, const void* k, const void* v, const void* bias, void* o, int H, int d,
                         int pair_order, int bias_prescaled, const BatchMeta& m, int* status, cudaStream_t st) {
  const __nv_bfloat16* qq = (const __nv_bfloat16*)q;
  const __nv_bfloat16* kk = (const __nv_bfloat16*)k;
  const __nv_bfloat16* vv = (const __nv_bfloat16*)v;
  const __nv_bfloat16* bb = (const __nv_bfloat16*)bias;
  __nv_bfloat16* oo = (__nv_bfloat16*)o;
  if (d == 16) return launch_attn<16>(qq, kk, vv, bb, oo, H, pair_order, bias_prescaled, m, status, st);
  if (d == 32) return launch_attn<32>(qq, kk, vv, bb, oo, H, pair_order, bias_prescaled, m, status, st);
  if (d == 64) return launch_attn<64>(qq, kk, vv, bb, oo, H, pair_order, bias_prescaled, m, status, st);
  return NT_ERR_UNSUPPORTED;
}

}  // namespace ntp
