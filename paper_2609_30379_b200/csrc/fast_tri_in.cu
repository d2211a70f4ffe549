// Triangle-update input projection on tcgen05 (bf16, float accumulate):
//   zh = LN(z);  a = sigmoid(zh W_ag^T) * (zh W_ap^T);  b = sigmoid(zh W_bg^T) * (zh W_bp^T)
// written channel-major (a[c][i][k], k contiguous) so the contraction's operands are K-major.
//
// LayerNorm is folded into the product: with W' = W * gamma (column scale, rounded to bf16),
// c1[n] = sum_k W'[n][k] and c0[n] = sum_k W[n][k] beta[k],
//   (LN(z) W^T)[n] = rstd * (z . W'[n] - mean * c1[n]) + c0[n],
// so the raw z tile goes from TMA straight into the MMA and only per-row mean / rstd (computed by
// the epilogue threads from the same shared-memory tile) are needed afterwards.
//
// A tile is 128 packed positions made of four 32-position chunks, each a run of consecutive k inside
// one pair row (s, i) taken from the offset table, so a warp's 32 accumulator rows are 32 consecutive
// k of one row and transpose into 64-byte channel-major runs.  The weights (4 c_h x c_z) stay
// resident in shared memory; the pair state is read exactly once.
#include <cstring>

#include "fast.cuh"
#include "tc_common.cuh"

namespace ntp {

constexpr int TI_CH = 32;                  // positions per chunk
constexpr int TI_THREADS = 64 + 128 + 256; // producer warp, MMA warp, 4 converter warps, 8 epilogue warps
constexpr int TI_MAXB = 16;

struct TriInParams {
  CUtensorMap zmap[TI_MAXB];               // {c_z, N (k), N (i)}, box {64, 32, 1}
  CUtensorMap wmap;                        // {c_z, 4 c_h}, box {64, 128}
  long long chunk_off[TI_MAXB + 1];
  long long cm_off[TI_MAXB];
  int N[TI_MAXB];
  int B, c_z, c_h;
  float eps;
  const float2* c01;                       // [4 c_h] (c0, c1)
  __nv_bfloat16* a;
  __nv_bfloat16* b;
  int* status;
};

__device__ inline bool ti_decode(const TriInParams& p, long long q, int& s, int& i, int& jc) {
  if (q >= p.chunk_off[p.B]) return false;
  s = 0;
  while (s + 1 < p.B && q >= p.chunk_off[s + 1]) ++s;
  const int cpr = (p.N[s] + TI_CH - 1) / TI_CH;
  const long long r = q - p.chunk_off[s];
  i = (int)(r / cpr);
  jc = (int)(r - (long long)i * cpr) * TI_CH;
  return true;
}

__device__ inline float sigmoid_fast(float x) {
  float t;
  asm("tanh.approx.f32 %0, %1;\n" : "=f"(t) : "f"(0.5f * x));
  return fmaf(0.5f, t, 0.5f);
}

__global__ void __launch_bounds__(TI_THREADS, 1) tri_in_kernel(const __grid_constant__ TriInParams p) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[11];
  __shared__ float2 sStats[2][128];        // per stage: (mean, rstd) of every tile row
  __shared__ unsigned tmem_base_s;
  __shared__ int abort_flag;
  unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
  const int c_z = p.c_z, c_h = p.c_h;
  const int nslab = c_z / 64;
  const int w_slab_bytes = 4 * c_h * 128;          // one 64-channel slab of all 4 c_h weight rows
  const int w_bytes = nslab * w_slab_bytes;
  const int a_slab_bytes = 128 * 128;
  const int a_stage_bytes = nslab * a_slab_bytes;
  unsigned char* sW = smem;
  unsigned char* sA = sW + w_bytes;                // 2 stages
  unsigned char* sStage = sA + 2 * a_stage_bytes;  // 8 warps x 2 KB transpose staging
  float2* sC = reinterpret_cast<float2*>(sStage + 8 * 2048);
  unsigned long long* afull = bars;        // [2]
  unsigned long long* aempty = bars + 2;   // [2]
  unsigned long long* tfull = bars + 4;    // [2]
  unsigned long long* tempty = bars + 6;   // [2]
  unsigned long long* wfull = bars + 8;
  unsigned long long* aconv = bars + 9;    // [2] tile converted to fp16, statistics published

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < 2; ++s) {
      mbar_init(&afull[s], 1);
      mbar_init(&aempty[s], 1 + 8);        // MMA commit + one arrival per epilogue warp
      mbar_init(&tfull[s], 1);
      mbar_init(&tempty[s], 8);
      mbar_init(&aconv[s], 4);
    }
    mbar_init(wfull, 1);
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&tmem_base_s, 512);
  for (int n = threadIdx.x; n < 4 * c_h; n += TI_THREADS) sC[n] = p.c01[n];
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = tmem_base_s;
  AbortCtx ab{p.status, &abort_flag};
  const long long nchunks = p.chunk_off[p.B];
  const long long ntiles = (nchunks + 3) / 4;
  const int Nu = 2 * c_h;                          // accumulator columns per unit (gate | value)

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ producer
    mbar_expect_tx(wfull, w_bytes);
    for (int sl = 0; sl < nslab; ++sl)
      for (int rb = 0; rb < 4 * c_h / 128; ++rb)
        tma_load_2d(sW + sl * w_slab_bytes + rb * 128 * 128, &p.wmap, wfull, sl * 64, rb * 128);
    int stage = 0;
    unsigned phase = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
      mbar_wait(&aempty[stage], phase ^ 1, ab);
      int nvalid = 0;
      for (int q = 0; q < 4; ++q) nvalid += (4 * t + q < nchunks) ? 1 : 0;
      mbar_expect_tx(&afull[stage], nvalid * nslab * TI_CH * 128);
      for (int q = 0; q < nvalid; ++q) {
        int s, i, jc;
        ti_decode(p, 4 * t + q, s, i, jc);
        for (int sl = 0; sl < nslab; ++sl)
          tma_load_4d(sA + stage * a_stage_bytes + sl * a_slab_bytes + q * TI_CH * 128, &p.zmap[s], &afull[stage],
                      sl * 64, jc, i, 0);
      }
      if (++stage == 2) { stage = 0; phase ^= 1; }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    mbar_wait(wfull, 0, ab);
    int stage = 0;
    unsigned phase = 0, tph[2] = {0, 0};
    long long unit = 0;
    const unsigned idesc = idesc_f16(128, Nu, 0, 0, FMT_F16, FMT_F16);   // z tile converted to fp16, folded weights fp16
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
      mbar_wait(&aconv[stage], phase, ab);
      tc_fence_after();
      const unsigned a_addr = smem_u32(sA + stage * a_stage_bytes);
      for (int u = 0; u < 2; ++u, ++unit) {
        const int buf = (int)(unit & 1);
        mbar_wait(&tempty[buf], tph[buf] ^ 1, ab);
        tph[buf] ^= 1;
        tc_fence_after();
        const unsigned d_tmem = tmem_base + buf * 256;
        for (int sl = 0; sl < nslab; ++sl) {
          const unsigned w_addr = smem_u32(sW + sl * w_slab_bytes + u * Nu * 128);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            umma_bf16(d_tmem, desc_kmajor_sw128(a_addr + sl * a_slab_bytes + k4 * 32),
                      desc_kmajor_sw128(w_addr + k4 * 32), idesc, (sl | k4) != 0);
        }
        tc_commit(&tfull[buf]);
      }
      tc_commit(&aempty[stage]);
      if (++stage == 2) { stage = 0; phase ^= 1; }
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------------ converters (4 warps, one row per thread)
    const int row = (warp - 2) * 32 + lane;
    int stage = 0;
    unsigned phase = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
      mbar_wait(&afull[stage], phase, ab);
      float sum, sq;
      convert_row_bf16_to_f16(sA + stage * a_stage_bytes, nslab, a_slab_bytes, row, sum, sq);
      const float mean = sum / (float)c_z;
      const float var = fmaxf(sq / (float)c_z - mean * mean, 0.f);
      sStats[stage][row] = make_float2(mean, rsqrtf(var + p.eps));
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&aconv[stage]);
      if (++stage == 2) { stage = 0; phase ^= 1; }
    }
  } else if (warp >= 6) {
    // ------------------------------------------------------------------ epilogue (8 warps)
    const int quarter = warp & 3;                  // TMEM lane quarter this warp may read
    const int half = (warp - 6) >> 2;              // which half of the channels this warp handles
    const int row = quarter * 32 + lane;           // accumulator row = position inside the tile
    unsigned char* stg = sStage + (warp - 6) * 2048;
    int stage = 0;
    unsigned phase = 0, tph[2] = {0, 0};
    long long unit = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x) {
      // chunk of this warp: quarter-th chunk of the tile
      int s = 0, i = 0, jc = 0;
      const bool valid = ti_decode(p, 4 * t + quarter, s, i, jc);
      mbar_wait(&aconv[stage], phase, ab);         // statistics of this tile are published
      const float2 stt = sStats[stage][row];
      __syncwarp();
      if (lane == 0) mbar_arrive(&aempty[stage]);
      const float mean = stt.x, rstd = stt.y;
      const int N = valid ? p.N[s] : 1;
      const int ld = round_up8(N);
      const long long plane = (long long)N * ld;
      for (int u = 0; u < 2; ++u, ++unit) {
        const int buf = (int)(unit & 1);
        mbar_wait(&tfull[buf], tph[buf], ab);
        tph[buf] ^= 1;
        tc_fence_after();
        const unsigned taddr = tmem_base + ((unsigned)(quarter * 32) << 16) + buf * 256;
        __nv_bfloat16* outp = (u == 0 ? p.a : p.b) + (valid ? (long long)c_h * p.cm_off[s] + (long long)i * ld + jc : 0);
        const float2* cg = sC + u * Nu;            // gate rows first, value rows c_h later
        for (int c0 = half * (c_h / 2); c0 < (half + 1) * (c_h / 2); c0 += 32) {
          unsigned rg[32], rv[32];
          tmem_ld32(taddr + c0, rg);
          tmem_ld32(taddr + c_h + c0, rv);
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 32; ++e) {
            const float2 kg = cg[c0 + e], kv = cg[c_h + c0 + e];
            const float xg = fmaf(rstd, __uint_as_float(rg[e]) - mean * kg.y, kg.x);
            const float xv = fmaf(rstd, __uint_as_float(rv[e]) - mean * kv.y, kv.x);
            const float val = fminf(fmaxf(sigmoid_fast(xg) * xv, -65504.f), 65504.f);
            reinterpret_cast<__half*>(stg)[e * 32 + lane] = __float2half_rn(val);
          }
          __syncwarp();
          if (valid) {
#pragma unroll
            for (int it = 0; it < 4; ++it) {
              const int cl = it * 8 + (lane >> 2), vec = lane & 3;
              if (jc + vec * 8 < ld) {
                const uint4 v = *reinterpret_cast<const uint4*>(stg + cl * 64 + vec * 16);
                *reinterpret_cast<uint4*>(outp + (long long)(c0 + cl) * plane + vec * 8) = v;
              }
            }
          }
          __syncwarp();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&tempty[buf]);
      }
      if (++stage == 2) { stage = 0; phase ^= 1; }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

bool fast_tri_in_supported(int c_z, int c_h) { return (c_z == 64 || c_z == 128) && (c_h == 64 || c_h == 128); }

nt_status fast_tri_in(const void* z, const TriPrep& tp, float eps, int c_z, int c_h, void* a, void* b,
                      const BatchMeta& m, int* status, cudaStream_t st) {
  const void* wprime = tp.w1;
  const float2* c01 = (const float2*)tp.c01_1;
  const int nslab = c_z / 64;
  const size_t smem = (size_t)nslab * 4 * c_h * 128 + 2 * (size_t)nslab * 128 * 128 + 8 * 2048 + 4 * c_h * 8 + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(tri_in_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
      return cuda_fail("tri_in smem attribute");
    attr_set = true;
  }
  for (int g0 = 0; g0 < m.B; g0 += TI_MAXB) {
    TriInParams p;
    memset(&p, 0, sizeof(p));
    p.B = m.B - g0 < TI_MAXB ? m.B - g0 : TI_MAXB;
    p.c_z = c_z;
    p.c_h = c_h;
    p.eps = eps;
    p.c01 = c01;
    p.a = (__nv_bfloat16*)a;
    p.b = (__nv_bfloat16*)b;
    p.status = status;
    {
      const unsigned long long dims[2] = {(unsigned long long)c_z, (unsigned long long)4 * c_h};
      const unsigned long long strides[1] = {(unsigned long long)c_z * 2};
      const unsigned box[2] = {64, 128};
      if (!make_tmap_bf16(&p.wmap, wprime, 2, dims, strides, box)) { fprintf(stderr, "libnested_pair: tensor map encode failed (%s:%d)\n", __FILE__, __LINE__); return NT_ERR_CUDA; }
    }
    p.chunk_off[0] = 0;
    for (int l = 0; l < TI_MAXB; ++l) {
      const int N = l < p.B ? m.N[g0 + l] : 0;
      p.N[l] = N;
      p.cm_off[l] = l < p.B ? m.cm_off[g0 + l] : 0;
      p.chunk_off[l + 1] = p.chunk_off[l] + (long long)N * ((N + TI_CH - 1) / TI_CH);
      if (N > 0) {
        const unsigned long long dims[4] = {(unsigned long long)c_z, (unsigned long long)N, (unsigned long long)N, 1};
        const unsigned long long strides[3] = {(unsigned long long)c_z * 2, (unsigned long long)N * c_z * 2,
                                               (unsigned long long)N * N * c_z * 2};
        const unsigned box[4] = {64, TI_CH, 1, 1};
        const char* base = (const char*)z + (size_t)m.pair_off[g0 + l] * c_z * 2;
        if (!make_tmap_bf16(&p.zmap[l], base, 4, dims, strides, box)) { fprintf(stderr, "libnested_pair: tensor map encode failed (%s:%d)\n", __FILE__, __LINE__); return NT_ERR_CUDA; }
      }
    }
    const long long ntiles = (p.chunk_off[p.B] + 3) / 4;
    if (ntiles == 0) continue;
    const unsigned grid = (unsigned)(ntiles < 148 ? ntiles : 148);
    {
      LaunchScope ls("tri_in", st);
      tri_in_kernel<<<grid, TI_THREADS, smem, st>>>(p);
    }
    if (cudaPeekAtLastError() != cudaSuccess) return cuda_fail("tensor-core kernel launch");
  }
  return NT_OK;
}

}  // namespace ntp
