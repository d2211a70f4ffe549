// Row-wise pair-biased attention core for bf16, head dims 16 / 32 / 64.
//
// One CTA (4 warps) owns 64 queries j of one (sample, head) and walks a chunk of attention rows i
// (pair order) or the single row of a sample (token order).  The bias tile bias[h][j0:j0+64][:] is
// the same for every row i of the sample, so it is fetched once per CTA and stays in shared memory
// while the CTA streams the rows' K / V blocks through a cp.async pipeline.  Scores and P.V run on
// the tensor cores (m16n8k16 bf16, P kept in registers between the two products); the softmax is
// the online (running max / running sum) form in float, in the log2 domain.
// The core is bound by the softmax arithmetic, not by the tensor pipe: per score element there
// are 2*d tensor flops against ~7 CUDA-core instructions and one exponential.
#include "fast.cuh"

namespace ntp {

constexpr int AT_Q = 64;          // queries per CTA
constexpr int AT_K = 64;          // keys per pipeline step
constexpr int AT_STAGES = 3;
constexpr int AT_THREADS = 128;
constexpr int AT_RES_CAP = 112 * 1024;   // largest resident bias tile (bytes)

__host__ __device__ inline int at_bias_stride(int N) {   // bytes per resident bias row: 16 mod 32
  int b = round_up8(N) * 2;
  return (b / 16) % 2 == 0 ? b + 16 : b;
}

__device__ inline void cp_async16(void* smem, const void* gmem, bool valid) {
  const unsigned sa = (unsigned)__cvta_generic_to_shared(smem);
  const int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(sa), "l"(gmem), "r"(sz));
}
__device__ inline void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ inline void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }

__device__ inline void ldsm_x4(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(a));
}
__device__ inline void ldsm_x2(unsigned& r0, unsigned& r1, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];\n" : "=r"(r0), "=r"(r1) : "r"(a));
}
__device__ inline void ldsm_x4_t(unsigned& r0, unsigned& r1, unsigned& r2, unsigned& r3, const void* p) {
  const unsigned a = (unsigned)__cvta_generic_to_shared(p);
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
__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;\n" : "=f"(y) : "f"(x));
  return y;
}

template <int D>
__global__ void __launch_bounds__(AT_THREADS)
attn_core_mma_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                     const __nv_bfloat16* __restrict__ v, const __nv_bfloat16* __restrict__ bias,
                     __nv_bfloat16* __restrict__ o, int H, int pair_order, int ichunk, int bias_bytes, BatchMeta m) {
  constexpr int ROWB = D * 2 + 16;              // padded K / V / Q row (bytes)
  constexpr int KV_STAGE = AT_K * ROWB;
  constexpr int BS_ROWB = AT_K * 2 + 16;        // streamed bias block row (bytes)
  constexpr int CH = D / 8;                     // 16-byte chunks per row
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* sK = smem;                                    // [STAGES][64][ROWB]
  unsigned char* sV = sK + AT_STAGES * KV_STAGE;               // [STAGES][64][ROWB]
  unsigned char* sQ = sV + AT_STAGES * KV_STAGE;               // [STAGES][64][ROWB], slot of the row's first step
  unsigned char* sB = sQ + AT_STAGES * AT_Q * ROWB;                    // resident tile or [STAGES][64][BS_ROWB]
  __shared__ int s_item[4];

  if (threadIdx.x == 0) {
    long long w = blockIdx.x;
    int s = 0;
    for (; s < m.B; ++s) {
      const int N = m.N[s];
      const long long njb = (N + AT_Q - 1) / AT_Q;
      const long long nic = pair_order ? (N + ichunk - 1) / ichunk : (N > 0 ? 1 : 0);
      const long long cnt = njb * H * nic;
      if (w < cnt) break;
      w -= cnt;
    }
    s_item[0] = s;
    if (s < m.B) {
      const int N = m.N[s];
      const int njb = (N + AT_Q - 1) / AT_Q;
      s_item[1] = (int)(w % njb);                 // j block
      s_item[2] = (int)((w / njb) % H);           // head
      s_item[3] = (int)(w / ((long long)njb * H)); // i chunk
    }
  }
  __syncthreads();
  const int s = s_item[0];
  if (s >= m.B) return;
  const int N = m.N[s], ld = round_up8(N);
  const int j0 = s_item[1] * AT_Q, h = s_item[2];
  const int i_begin = pair_order ? s_item[3] * ichunk : 0;
  const int i_end = pair_order ? min(N, i_begin + ichunk) : 1;
  const int Hd = H * D;
  const int nkb = (N + AT_K - 1) / AT_K;
  const int steps = (i_end - i_begin) * nkb;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
  const bool has_bias = bias != nullptr;
  const int bstride = at_bias_stride(N);
  const bool resident = has_bias && AT_Q * bstride <= bias_bytes && AT_Q * bstride <= AT_RES_CAP;
  const __nv_bfloat16* bias_h = has_bias ? bias + (long long)H * m.cm_off[s] + (long long)h * N * ld : nullptr;

  auto row_base = [&](int i) -> long long {
    return pair_order ? m.pair_off[s] + (long long)i * N : m.tok_off[s];
  };

  // ---- resident bias tile: rows j0..j0+63, all keys
  if (resident) {
    const int chunks = ld / 8;
    for (int idx = tid; idx < AT_Q * chunks; idx += AT_THREADS) {
      const int r = idx / chunks, c = idx - r * chunks;
      const bool ok = j0 + r < N;
      const __nv_bfloat16* src = bias_h + (long long)(ok ? j0 + r : 0) * ld + c * 8;
      cp_async16(sB + r * bstride + c * 16, src, ok);
    }
  }

  auto issue = [&](int t) {   // loads of pipeline step t into slot t % STAGES
    if (t < steps) {
      const int i = i_begin + t / nkb, kb = t - (t / nkb) * nkb;
      const int slot = t % AT_STAGES;
      const long long base = row_base(i);
      const int k0 = kb * AT_K;
      for (int idx = tid; idx < AT_K * CH; idx += AT_THREADS) {
        const int r = idx / CH, c = idx - r * CH;
        const bool ok = k0 + r < N;
        const long long off = (base + (ok ? k0 + r : 0)) * Hd + h * D + c * 8;
        cp_async16(sK + slot * KV_STAGE + r * ROWB + c * 16, k + off, ok);
        cp_async16(sV + slot * KV_STAGE + r * ROWB + c * 16, v + off, ok);
      }
      if (kb == 0) {
        unsigned char* dst = sQ + slot * AT_Q * ROWB;
        for (int idx = tid; idx < AT_Q * CH; idx += AT_THREADS) {
          const int r = idx / CH, c = idx - r * CH;
          const bool ok = j0 + r < N;
          cp_async16(dst + r * ROWB + c * 16, q + (base + (ok ? j0 + r : 0)) * Hd + h * D + c * 8, ok);
        }
      }
      if (has_bias && !resident) {
        unsigned char* dst = sB + slot * AT_Q * BS_ROWB;
        for (int idx = tid; idx < AT_Q * (AT_K / 8); idx += AT_THREADS) {
          const int r = idx / (AT_K / 8), c = idx - r * (AT_K / 8);
          const bool ok = j0 + r < N && k0 + c * 8 < ld;
          const __nv_bfloat16* src = bias_h + (long long)(ok ? j0 + r : 0) * ld + (ok ? k0 + c * 8 : 0);
          cp_async16(dst + r * BS_ROWB + c * 16, src, ok);
        }
      }
    }
    cp_async_commit();
  };

#pragma unroll
  for (int t = 0; t < AT_STAGES - 1; ++t) issue(t);

  const float sc2 = rsqrtf((float)D) * 1.4426950408889634f;
  const float l2e = 1.4426950408889634f;
  const bool warp_active = j0 + warp * 16 < N;
  unsigned qf[D / 16][4];
  float oacc[D / 8][4];
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};

  for (int t = 0; t < steps; ++t) {
    cp_async_wait<AT_STAGES - 2>();
    __syncthreads();
    issue(t + AT_STAGES - 1);
    if (!warp_active) continue;
    const int irel = t / nkb, kb = t - irel * nkb;
    const int slot = t % AT_STAGES;
    const int k0 = kb * AT_K;
    if (kb == 0) {
      const unsigned char* qs = sQ + slot * AT_Q * ROWB;
#pragma unroll
      for (int ks = 0; ks < D / 16; ++ks) {
        const int mtx = lane >> 3;
        const int row = warp * 16 + (mtx & 1) * 8 + (lane & 7);
        const int col = ks * 16 + (mtx >> 1) * 8;
        ldsm_x4(qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3], qs + row * ROWB + col * 2);
      }
#pragma unroll
      for (int nd = 0; nd < D / 8; ++nd) oacc[nd][0] = oacc[nd][1] = oacc[nd][2] = oacc[nd][3] = 0.f;
      mrow[0] = mrow[1] = -INFINITY;
      lrow[0] = lrow[1] = 0.f;
    }
    // ---- S = Q K^T for 16 queries x 64 keys
    float sacc[AT_K / 8][4];
    const unsigned char* ks_ = sK + slot * KV_STAGE;
#pragma unroll
    for (int nt = 0; nt < AT_K / 8; ++nt) {
      sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
      if constexpr (D == 16) {
        unsigned b0, b1;
        ldsm_x2(b0, b1, ks_ + (nt * 8 + (lane & 7)) * ROWB + ((lane >> 3) & 1) * 16);
        mma_bf16(sacc[nt], qf[0], b0, b1);
      } else {
#pragma unroll
        for (int kp = 0; kp < D / 32; ++kp) {
          unsigned b0, b1, b2, b3;
          ldsm_x4(b0, b1, b2, b3, ks_ + (nt * 8 + (lane & 7)) * ROWB + (kp * 4 + (lane >> 3)) * 16);
          mma_bf16(sacc[nt], qf[kp * 2], b0, b1);
          mma_bf16(sacc[nt], qf[kp * 2 + 1], b2, b3);
        }
      }
    }
    // ---- scale, bias, mask, online softmax
    const unsigned char* brow0 = nullptr;
    const unsigned char* brow1 = nullptr;
    if (has_bias) {
      if (resident) {
        brow0 = sB + (warp * 16 + g) * bstride + k0 * 2;
        brow1 = brow0 + 8 * bstride;
      } else {
        brow0 = sB + slot * AT_Q * BS_ROWB + (warp * 16 + g) * BS_ROWB;
        brow1 = brow0 + 8 * BS_ROWB;
      }
    }
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < AT_K / 8; ++nt) {
      const int kc = nt * 8 + 2 * tq;
      float b00 = 0.f, b01 = 0.f, b10 = 0.f, b11 = 0.f;
      if (has_bias && k0 + kc < ld) {
        const unsigned w0 = *reinterpret_cast<const unsigned*>(brow0 + kc * 2);
        const unsigned w1 = *reinterpret_cast<const unsigned*>(brow1 + kc * 2);
        b00 = __uint_as_float(w0 << 16); b01 = __uint_as_float(w0 & 0xffff0000u);
        b10 = __uint_as_float(w1 << 16); b11 = __uint_as_float(w1 & 0xffff0000u);
      }
      const bool v0 = k0 + kc < N, v1 = k0 + kc + 1 < N;
      sacc[nt][0] = v0 ? fmaf(sacc[nt][0], sc2, b00 * l2e) : -INFINITY;
      sacc[nt][1] = v1 ? fmaf(sacc[nt][1], sc2, b01 * l2e) : -INFINITY;
      sacc[nt][2] = v0 ? fmaf(sacc[nt][2], sc2, b10 * l2e) : -INFINITY;
      sacc[nt][3] = v1 ? fmaf(sacc[nt][3], sc2, b11 * l2e) : -INFINITY;
      mx0 = fmaxf(mx0, fmaxf(sacc[nt][0], sacc[nt][1]));
      mx1 = fmaxf(mx1, fmaxf(sacc[nt][2], sacc[nt][3]));
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float mn0 = fmaxf(mrow[0], mx0), mn1 = fmaxf(mrow[1], mx1);   // finite: key k0 is valid
    const float cr0 = fast_exp2(mrow[0] - mn0), cr1 = fast_exp2(mrow[1] - mn1);
    mrow[0] = mn0;
    mrow[1] = mn1;
    float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
    for (int nt = 0; nt < AT_K / 8; ++nt) {
      sacc[nt][0] = fast_exp2(sacc[nt][0] - mn0);
      sacc[nt][1] = fast_exp2(sacc[nt][1] - mn0);
      sacc[nt][2] = fast_exp2(sacc[nt][2] - mn1);
      sacc[nt][3] = fast_exp2(sacc[nt][3] - mn1);
      ps0 += sacc[nt][0] + sacc[nt][1];
      ps1 += sacc[nt][2] + sacc[nt][3];
    }
    lrow[0] = lrow[0] * cr0 + ps0;
    lrow[1] = lrow[1] * cr1 + ps1;
#pragma unroll
    for (int nd = 0; nd < D / 8; ++nd) {
      oacc[nd][0] *= cr0; oacc[nd][1] *= cr0;
      oacc[nd][2] *= cr1; oacc[nd][3] *= cr1;
    }
    // ---- O += P V
    const unsigned char* vs_ = sV + slot * KV_STAGE;
#pragma unroll
    for (int kk = 0; kk < AT_K / 16; ++kk) {
      unsigned pf[4];
      pf[0] = pack_bf16(sacc[2 * kk][0], sacc[2 * kk][1]);
      pf[1] = pack_bf16(sacc[2 * kk][2], sacc[2 * kk][3]);
      pf[2] = pack_bf16(sacc[2 * kk + 1][0], sacc[2 * kk + 1][1]);
      pf[3] = pack_bf16(sacc[2 * kk + 1][2], sacc[2 * kk + 1][3]);
#pragma unroll
      for (int np = 0; np < D / 16; ++np) {
        const int mtx = lane >> 3;
        const int krow = kk * 16 + (mtx & 1) * 8 + (lane & 7);
        const int dcol = (np * 2 + (mtx >> 1)) * 8;
        unsigned b0, b1, b2, b3;
        ldsm_x4_t(b0, b1, b2, b3, vs_ + krow * ROWB + dcol * 2);
        mma_bf16(oacc[np * 2], pf, b0, b1);
        mma_bf16(oacc[np * 2 + 1], pf, b2, b3);
      }
    }
    // ---- last key block of this row: normalise and store
    if (kb == nkb - 1) {
      float l0 = lrow[0], l1 = lrow[1];
      l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
      l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
      l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
      const float inv0 = 1.0f / l0, inv1 = 1.0f / l1;
      const long long base = row_base(i_begin + irel);
      const int r0 = j0 + warp * 16 + g, r1 = r0 + 8;
#pragma unroll
      for (int nd = 0; nd < D / 8; ++nd) {
        const int col = h * D + nd * 8 + 2 * tq;
        if (r0 < N)
          *reinterpret_cast<unsigned*>(o + (base + r0) * Hd + col) = pack_bf16(oacc[nd][0] * inv0, oacc[nd][1] * inv0);
        if (r1 < N)
          *reinterpret_cast<unsigned*>(o + (base + r1) * Hd + col) = pack_bf16(oacc[nd][2] * inv1, oacc[nd][3] * inv1);
      }
    }
  }
  cp_async_wait<0>();
}

bool fast_attn_core_supported(int H, int d) { return (d == 16 || d == 32 || d == 64) && H >= 1; }

template <int D>
static nt_status launch_attn_mma(const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                 const __nv_bfloat16* bias, __nv_bfloat16* o, int H, int pair_order,
                                 const BatchMeta& m, cudaStream_t st) {
  constexpr int ROWB = D * 2 + 16;
  long long rows_i = 0;
  int bias_bytes = 0;
  for (int s = 0; s < m.B; ++s) {
    rows_i += pair_order ? m.N[s] : 1;
    if (bias) {
      const int res = AT_Q * at_bias_stride(m.N[s]);
      const int need = res <= AT_RES_CAP ? res : AT_STAGES * AT_Q * (AT_K * 2 + 16);
      if (need > bias_bytes) bias_bytes = need;
    }
  }
  int ichunk = 16;
  auto count = [&](int ic) {
    long long c = 0;
    for (int s = 0; s < m.B; ++s) {
      const long long N = m.N[s], njb = (N + AT_Q - 1) / AT_Q;
      const long long nic = pair_order ? (N + ic - 1) / ic : (N > 0 ? 1 : 0);
      c += njb * H * nic;
    }
    return c;
  };
  if (pair_order && count(ichunk) < 148 * 6) ichunk = 8;
  if (pair_order && count(ichunk) < 148 * 6) ichunk = 4;
  const long long blocks = count(ichunk);
  if (blocks == 0) return NT_OK;
  if (blocks > 0x7FFFFFFFll) return NT_ERR_UNSUPPORTED;
  const size_t smem = (size_t)2 * AT_STAGES * AT_K * ROWB + AT_STAGES * AT_Q * ROWB + bias_bytes;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(attn_core_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) !=
        cudaSuccess)
      return cuda_fail("shared memory attribute");
    attr_set = true;
  }
  {
    LaunchScope ls("attn_core", st);
    attn_core_mma_kernel<D><<<(unsigned)blocks, AT_THREADS, smem, st>>>(q, k, v, bias, o, H, pair_order, ichunk,
                                                                       bias_bytes, m);
  }
  return cuda_ok();
}

nt_status fast_attn_core(const void* q, const void* k, const void* v, const void* bias, void* o, int H, int d,
                         int pair_order, const BatchMeta& m, cudaStream_t st) {
  const __nv_bfloat16* qq = (const __nv_bfloat16*)q;
  const __nv_bfloat16* kk = (const __nv_bfloat16*)k;
  const __nv_bfloat16* vv = (const __nv_bfloat16*)v;
  const __nv_bfloat16* bb = (const __nv_bfloat16*)bias;
  __nv_bfloat16* oo = (__nv_bfloat16*)o;
  if (d == 16) return launch_attn_mma<16>(qq, kk, vv, bb, oo, H, pair_order, m, st);
  if (d == 32) return launch_attn_mma<32>(qq, kk, vv, bb, oo, H, pair_order, m, st);
  if (d == 64) return launch_attn_mma<64>(qq, kk, vv, bb, oo, H, pair_order, m, st);
  return NT_ERR_UNSUPPORTED;
}

}  // namespace ntp
