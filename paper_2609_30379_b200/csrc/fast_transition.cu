// SwiGLU pair transition on tcgen05, fused so that the expanded hidden activation never leaves the SM:
//   zh = LN(z);  z += (silu(zh W_a^T) * (zh W_b^T)) W_2^T          (position-wise on packed rows)
//
// A persistent CTA per SM walks tiles of 128 consecutive packed rows.  The hidden width is processed in chunks of 64
// units; per chunk
//   GEMM 1  [128 rows x c] x [64 gate rows | 64 value rows of the folded W_a / W_b]^T -> 128 TMEM columns
//   gate    h = silu(g) * v in registers (g arrives halved: silu(g) = g' tanh(g') + g' with g' = g / 2), written as
//           a bf16 K-major tile into shared memory
//   GEMM 2  out[128 rows x c] += h[128 x 64] x W_2[:, chunk]^T, accumulated over the chunks in TMEM
// and at the end of the tile out + z goes back through the z tile in shared memory and TMA stores.
// LayerNorm is folded into the weights (W' = W gamma, fp16); its mean term rides in GEMM 1 as one more K step
// ((-mean_hi, -mean_lo, -mean_hi) per row against (c1_hi, c1_hi, c1_lo) per weight row), rstd and c0 are applied in
// the gate stage; the z tile itself is only converted bf16 -> fp16 (exact), because it is also the residual.
// The weights do not fit in shared memory (3 c hidden elements): every chunk's W_a, W_b, W_2 slices stream from L2
// through a two-stage ring.  The kernel is bound by the tensor pipe (6 c hidden flops per row).
// Roles: warp 0 TMA producer, warp 1 MMA issuer (converged, one elected lane), warps 2-5 converters (one row per
// thread: statistics, fp16 copy, augmentation columns), warps 6-13 gate stage and output stage (two per TMEM lane
// quarter).  All waits are bounded.
#include <cstring>

#include "fast.cuh"
#include "tc_common.cuh"

namespace ntp {

constexpr int TR_THREADS = 64 + 128 + 256;
constexpr int TR_CHUNK = 64;                 // hidden units per chunk

struct TransParams {
  CUtensorMap zmap;      // state {c, rows}, box {64, 128} (loads)
  CUtensorMap zsmap;     // same tensor, box {64, 32} (stores, one per epilogue warp)
  CUtensorMap w1map;     // folded [W_a / 2; W_b] {c, 2 hidden} fp16, box {64, 64}
  CUtensorMap w1xmap;    // augmentation columns {8, 2 * 2 hidden} fp16, box {8, 64}, no swizzle
  CUtensorMap w2map;     // W_2 {hidden, c} bf16, box {64, c}
  const float2* c01;     // [2 hidden] (c0, c1) of the folded rows
  long long rows;
  int c, hidden;
  float eps;
  int* status;
};

__device__ inline float tr_tanh(float x) {
  float t;
  asm("tanh.approx.f32 %0, %1;\n" : "=f"(t) : "f"(x));
  return t;
}

__global__ void __launch_bounds__(TR_THREADS, 1) transition_kernel(const __grid_constant__ TransParams p) {
  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[22];
  __shared__ float sRstd[2][128];
  __shared__ unsigned tmem_base_s;
  __shared__ int abort_flag;
  unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
  const int c = p.c, hidden = p.hidden;
  const int nslab = c / 64, nchunk = hidden / TR_CHUNK;
  const int slab = 128 * 128;                        // [128 rows][64 channels] of 16-bit elements
  const int z_stage = nslab * slab;
  const int w1_bytes = nslab * slab;                 // 128 weight rows (64 gate | 64 value) x c
  const int w2_bytes = c * 128;                      // c rows x 64 hidden units
  const int w_stage = w1_bytes + w2_bytes + 2048;    // + augmentation columns 0-7 of the 128 weight rows
  unsigned char* sZ = smem;                          // 2 stages
  unsigned char* sW = sZ + 2 * z_stage;              // 2 stages: [W1 chunk | W2 chunk | W1 augmentation]
  unsigned char* sH = sW + 2 * w_stage;              // 2 buffers of the bf16 hidden chunk [128 rows][64]
  unsigned char* sZx = sH + 2 * slab;                // 2 stages x [128][8] fp16: augmentation columns 0-7 of the rows
  unsigned char* sZero = sZx + 2 * 2048;             // [128][8] zeros: augmentation columns 8-15 of either operand
  float* sC0 = reinterpret_cast<float*>(sZero + 2048);   // c0 of the gate rows [hidden], then of the value rows [hidden]
  unsigned long long* zfull = bars;        // [2]
  unsigned long long* zempty = bars + 2;   // [2] the tile's stores have read the stage
  unsigned long long* zconv = bars + 4;    // [2]
  unsigned long long* wfull = bars + 6;    // [2]
  unsigned long long* wempty = bars + 8;   // [2]
  unsigned long long* gvfull = bars + 10;  // [2] gate | value accumulators of a chunk are complete
  unsigned long long* gvempty = bars + 12; // [2]
  unsigned long long* hfull = bars + 14;   // [2] hidden chunk written
  unsigned long long* hempty = bars + 16;  // [2]
  unsigned long long* ofull = bars + 18;   // [2] output accumulator of a tile is complete
  unsigned long long* oempty = bars + 20;  // [2]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < 2; ++s) {
      mbar_init(&zfull[s], 1);
      mbar_init(&zempty[s], 4 * nslab);
      mbar_init(&zconv[s], 4);
      mbar_init(&wfull[s], 1);
      mbar_init(&wempty[s], 1);
      mbar_init(&gvfull[s], 1);
      mbar_init(&gvempty[s], 8);
      mbar_init(&hfull[s], 8);
      mbar_init(&hempty[s], 1);
      mbar_init(&ofull[s], 1);
      mbar_init(&oempty[s], 8);
    }
    mbar_fence_init();
  }
  if (warp == 1) tmem_alloc(&tmem_base_s, 512);
  for (int n = threadIdx.x; n < 2 * hidden; n += TR_THREADS) sC0[n] = p.c01[n].x;
  for (int idx = threadIdx.x; idx < (2 * 2048 + 2048) / 16; idx += TR_THREADS)      // augmentation tiles start as zeros
    *reinterpret_cast<uint4*>(sZx + idx * 16) = make_uint4(0, 0, 0, 0);
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem_base = tmem_base_s;
  AbortCtx ab{p.status, &abort_flag};
  const long long ntiles = (p.rows + 127) / 128;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer: lane l issues load l of a group
    unsigned gq = 0;
    int tn = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, ++tn) {
      const int zs = tn & 1;
      if (lane == 0) {
        mbar_wait(&zempty[zs], ((tn >> 1) & 1) ^ 1, ab);
        mbar_expect_tx(&zfull[zs], z_stage);
      }
      __syncwarp();
      if (lane < nslab) tma_load_2d(sZ + zs * z_stage + lane * slab, &p.zmap, &zfull[zs], lane * 64, (int)(t * 128));
      for (int q = 0; q < nchunk; ++q, ++gq) {
        const unsigned ws = gq & 1;
        unsigned char* wst = sW + ws * w_stage;
        if (lane == 0) {
          mbar_wait(&wempty[ws], ((gq >> 1) & 1) ^ 1, ab);
          mbar_expect_tx(&wfull[ws], w_stage);
        }
        __syncwarp();
        // W1 chunk: rows 0-63 = gate rows q * 64 .., rows 64-127 = value rows hidden + q * 64 ..; per 64-channel slab
        if (lane < 2 * nslab) {
          const int sl = lane >> 1, part = lane & 1;
          tma_load_2d(wst + sl * slab + part * 64 * 128, &p.w1map, &wfull[ws], sl * 64, part * hidden + q * TR_CHUNK);
        } else if (lane < 2 * nslab + 2) {
          const int part = lane - 2 * nslab;      // augmentation columns 0-7 of the same rows (region 0 of the table)
          tma_load_2d(wst + w1_bytes + w2_bytes + part * 64 * 16, &p.w1xmap, &wfull[ws], 0, part * hidden + q * TR_CHUNK);
        } else if (lane == 2 * nslab + 2) {
          tma_load_2d(wst + w1_bytes, &p.w2map, &wfull[ws], q * TR_CHUNK, 0);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (whole warp, one elected lane issues)
    const unsigned idesc1 = idesc_f16(128, 128, 0, 0, FMT_F16, FMT_F16);     // rows x (64 gate | 64 value)
    const unsigned idesc2 = idesc_f16(128, c, 0, 0, FMT_BF16, FMT_BF16);     // rows x c, A = hidden chunk, B = W_2 slice
    const unsigned zero_addr = smem_u32(sZero);
    unsigned gq = 0;
    int tn = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, ++tn) {
      const int zs = tn & 1, ob = tn & 1;
      mbar_wait(&zconv[zs], (tn >> 1) & 1, ab);
      mbar_wait(&oempty[ob], ((tn >> 1) & 1) ^ 1, ab);
      tc_fence_after();
      const unsigned long long z_desc = desc_kmajor_sw128(smem_u32(sZ + zs * z_stage));
      const unsigned zx_addr = smem_u32(sZx + zs * 2048);
      const unsigned long long zx_desc = desc_kmajor_nosw(zx_addr, zero_addr - zx_addr, 128);
      const unsigned d_out = tmem_base + 256 + ob * 128;
      for (int q = 0; q <= nchunk; ++q) {
        if (q < nchunk) {
          const unsigned g = gq + q, ws = g & 1, gb = g & 1;
          mbar_wait(&wfull[ws], (g >> 1) & 1, ab);
          mbar_wait(&gvempty[gb], ((g >> 1) & 1) ^ 1, ab);
          tc_fence_after();
          const unsigned w_addr = smem_u32(sW + ws * w_stage);
          const unsigned long long w1_desc = desc_kmajor_sw128(w_addr);
          const unsigned wx_addr = w_addr + w1_bytes + w2_bytes;
          const unsigned d_gv = tmem_base + gb * 128;
#pragma unroll
          for (int sl = 0; sl < 2; ++sl)
            if (sl < nslab) {
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4)
                if (elect_one())
                  umma_bf16(d_gv, z_desc + (sl * (slab >> 4) + k4 * 2), w1_desc + (sl * (slab >> 4) + k4 * 2), idesc1, (sl | k4) != 0);
            }
          if (elect_one()) {
            umma_bf16(d_gv, zx_desc, desc_kmajor_nosw(wx_addr, zero_addr - wx_addr, 128), idesc1, 1);   // mean term
            tc_commit(&gvfull[gb]);
          }
          __syncwarp();
        }
        if (q >= 1) {
          const unsigned g = gq + q - 1, ws = g & 1, hb = g & 1;
          mbar_wait(&hfull[hb], (g >> 1) & 1, ab);
          tc_fence_after();
          const unsigned long long h_desc = desc_kmajor_sw128(smem_u32(sH + hb * slab));
          const unsigned long long w2_desc = desc_kmajor_sw128(smem_u32(sW + ws * w_stage) + w1_bytes);
#pragma unroll
          for (int k4 = 0; k4 < 4; ++k4)
            if (elect_one()) umma_bf16(d_out, h_desc + k4 * 2, w2_desc + k4 * 2, idesc2, (q - 1) != 0 || k4 != 0);
          if (elect_one()) {
            tc_commit(&hempty[hb]);
            tc_commit(&wempty[ws]);
            if (q == nchunk) tc_commit(&ofull[ob]);
          }
          __syncwarp();
        }
      }
      gq += nchunk;
    }
  } else if (warp >= 2 && warp < 6) {
    // ------------------------------------------------------------------ converters (4 warps, one row per thread)
    const int row = (warp - 2) * 32 + lane;
    int tn = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, ++tn) {
      const int zs = tn & 1;
      mbar_wait(&zfull[zs], (tn >> 1) & 1, ab);
      float sum, sq;
      convert_row_bf16_to_f16(sZ + zs * z_stage, nslab, slab, row, sum, sq);
      const float mean = sum / (float)c;
      sRstd[zs][row] = rsqrtf(fmaxf(sq / (float)c - mean * mean, 0.f) + p.eps);
      const __half zh = __float2half_rn(-mean), zl = __float2half_rn(-mean - __half2float(zh));
      __half2 p0 = __halves2half2(zh, zl), p1 = __halves2half2(zh, __float2half_rn(0.f));
      *reinterpret_cast<uint2*>(sZx + zs * 2048 + row * 16) = make_uint2(*reinterpret_cast<unsigned*>(&p0), *reinterpret_cast<unsigned*>(&p1));
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(&zconv[zs]);
    }
  } else {
    // ------------------------------------------------------------------ gate stage and output stage (8 warps)
    const int quarter = warp & 3, half = (warp - 6) >> 2;
    const int row = quarter * 32 + lane;
    const unsigned t_lane = tmem_base + ((unsigned)(quarter * 32) << 16);
    unsigned gq = 0;
    int tn = 0;
    for (long long t = blockIdx.x; t < ntiles; t += gridDim.x, ++tn) {
      const int zs = tn & 1, ob = tn & 1;
      float rstd = 0.f;
      for (int q = 0; q < nchunk; ++q) {
        const unsigned g = gq + q, gb = g & 1;
        mbar_wait(&gvfull[gb], (g >> 1) & 1, ab);      // GEMM 1 of this tile has run, so the converters' statistics are published
        tc_fence_after();
        if (q == 0) rstd = sRstd[zs][row];
        unsigned rg[32], rv[32];
        tmem_ld32(t_lane + gb * 128 + half * 32, rg);
        tmem_ld32(t_lane + gb * 128 + 64 + half * 32, rv);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&gvempty[gb]);
        const float* cg = sC0 + q * TR_CHUNK + half * 32;
        const float* cv = sC0 + hidden + q * TR_CHUNK + half * 32;
        unsigned w[16];
#pragma unroll
        for (int e = 0; e < 16; ++e) {
          const float2 kg = *reinterpret_cast<const float2*>(cg + 2 * e), kv = *reinterpret_cast<const float2*>(cv + 2 * e);
          const float g0 = fmaf(rstd, __uint_as_float(rg[2 * e]), kg.x), g1 = fmaf(rstd, __uint_as_float(rg[2 * e + 1]), kg.y);
          const float v0 = fmaf(rstd, __uint_as_float(rv[2 * e]), kv.x), v1 = fmaf(rstd, __uint_as_float(rv[2 * e + 1]), kv.y);
          // g arrives halved: silu(2 g') = g' tanh(g') + g'
          const float h0 = fmaf(g0, tr_tanh(g0), g0) * v0, h1 = fmaf(g1, tr_tanh(g1), g1) * v1;
          __nv_bfloat162 hh = __floats2bfloat162_rn(h0, h1);
          w[e] = *reinterpret_cast<unsigned*>(&hh);
        }
        mbar_wait(&hempty[gb], ((g >> 1) & 1) ^ 1, ab);  // GEMM 2 of the chunk two back has read this buffer
        unsigned char* hb = sH + gb * slab;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          *reinterpret_cast<uint4*>(hb + sw128_off(row, half * 4 + j)) = make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&hfull[gb]);
      }
      gq += nchunk;
      // ---- output stage: out + z through the z tile, then one TMA store per warp
      mbar_wait(&ofull[ob], (tn >> 1) & 1, ab);
      tc_fence_after();
      unsigned char* zt = sZ + zs * z_stage;
      const int cpw = c / 2;                              // channels per thread
      for (int c0 = half * cpw; c0 < (half + 1) * cpw; c0 += 32) {
        unsigned r[32];
        tmem_ld32(t_lane + 256 + ob * 128 + c0, r);
        tmem_ld_wait();
        unsigned char* zp = zt + (c0 >> 6) * slab;
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint4* ptr = reinterpret_cast<uint4*>(zp + sw128_off(row, ((c0 & 63) >> 3) + ch));
          const uint4 v = *ptr;
          unsigned wz[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 zo = unpack_h2(wz[e]);           // the tile holds the exact fp16 copy of z
            __nv_bfloat162 hh = __floats2bfloat162_rn(__uint_as_float(r[ch * 8 + 2 * e]) + zo.x, __uint_as_float(r[ch * 8 + 2 * e + 1]) + zo.y);
            wz[e] = *reinterpret_cast<unsigned*>(&hh);
          }
          *ptr = make_uint4(wz[0], wz[1], wz[2], wz[3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&oempty[ob]);
      fence_proxy_async_smem();
      if (nslab == 1) named_bar_sync(2 + quarter, 64);    // the two warps of a lane quarter share the only slab
      else __syncwarp();
      if (lane == 0 && (nslab == 2 || half == 0)) {
        const long long r0 = t * 128 + quarter * 32;
        if (r0 < p.rows) tma_store_2d(&p.zsmap, zt + (nslab == 2 ? half : 0) * slab + quarter * 32 * 128, (nslab == 2 ? half : 0) * 64, (int)r0);
        tma_store_commit();
        tma_store_wait_read0();
        mbar_arrive(&zempty[zs]);
      }
    }
    if (lane == 0) tma_store_wait_all0();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

bool fast_transition_supported(int c, int hidden) { return (c == 64 || c == 128) && hidden % TR_CHUNK == 0 && hidden >= TR_CHUNK && hidden <= 1024; }

nt_status fast_transition(void* z, const nt_transition_weights* W, float eps, int c, int hidden, long long rows,
                          void* prep, int* status, cudaStream_t st) {
  if (rows > 0x7FFFFF00ll) return NT_ERR_UNSUPPORTED;
  TransPrep tp{};
  nt_status r0 = fast_transition_prep(W, c, hidden, prep, tp, st);
  if (r0 != NT_OK) return r0;
  const int nslab = c / 64;
  const size_t smem = 2 * (size_t)nslab * 16384 + 2 * ((size_t)nslab * 16384 + (size_t)c * 128 + 2048) + 2 * 16384 + 3 * 2048 +
                      2 * (size_t)hidden * 4 + 1024;
  static bool attr_set = false;
  if (!attr_set) {
    if (cudaFuncSetAttribute(transition_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024) != cudaSuccess)
      return cuda_fail("transition smem attribute");
    attr_set = true;
  }
  if (smem > 225 * 1024) return NT_ERR_UNSUPPORTED;
  TransParams p;
  memset(&p, 0, sizeof(p));
  p.c01 = (const float2*)tp.c01;
  p.rows = rows;
  p.c = c;
  p.hidden = hidden;
  p.eps = eps;
  p.status = status;
  {
    const unsigned long long dims[2] = {(unsigned long long)c, (unsigned long long)rows};
    const unsigned long long strides[1] = {(unsigned long long)c * 2};
    const unsigned box[2] = {64, 128}, sbox[2] = {64, 32};
    if (!make_tmap_bf16(&p.zmap, z, 2, dims, strides, box)) return cuda_fail("transition z map");
    if (!make_tmap_bf16(&p.zsmap, z, 2, dims, strides, sbox)) return cuda_fail("transition z store map");
    const unsigned long long wdims[2] = {(unsigned long long)c, (unsigned long long)2 * hidden};
    const unsigned wbox[2] = {64, 64};
    if (!make_tmap_bf16(&p.w1map, tp.w1, 2, wdims, strides, wbox)) return cuda_fail("transition W1 map");
    const unsigned long long xdims[2] = {8, (unsigned long long)2 * tp.rows};
    const unsigned long long xstr[1] = {16};
    const unsigned xbox[2] = {8, 64};
    if (!make_tmap_16bit(&p.w1xmap, tp.aug, 2, xdims, xstr, xbox, 0)) return cuda_fail("transition augmentation map");
    const unsigned long long w2dims[2] = {(unsigned long long)hidden, (unsigned long long)c};
    const unsigned long long w2str[1] = {(unsigned long long)hidden * 2};
    const unsigned w2box[2] = {64, (unsigned)c};
    if (!make_tmap_bf16(&p.w2map, W->W_2, 2, w2dims, w2str, w2box)) return cuda_fail("transition W2 map");
  }
  const long long ntiles = (rows + 127) / 128;
  const unsigned grid = (unsigned)(ntiles < 148 ? ntiles : 148);
  {
    LaunchScope ls("transition", st);
    transition_kernel<<<grid, TR_THREADS, smem, st>>>(p);
  }
  return cuda_ok("transition launch");
}

}  // namespace ntp
