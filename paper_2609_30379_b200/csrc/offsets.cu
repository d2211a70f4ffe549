// nt_offsets_build: exclusive prefix sums of N_s and N_s^2, level-2 row splits and the
// position -> (sample, i, j) decode with the rows/columns gather maps (Sec. 3.1, Fig. 2, Eq. 3).
// Integer-only, CUDA cores; the decode is a pure streaming write of 28 bytes per position.
#include "common.cuh"

namespace ntp {

constexpr int SCAN_THREADS = 1024;

__global__ void __launch_bounds__(SCAN_THREADS)
scan_lengths_kernel(const int64_t* __restrict__ len, int B, long long T1, long long T2,
                    int64_t* __restrict__ tok_off, int64_t* __restrict__ pair_off, int32_t* status) {
  __shared__ long long s1[SCAN_THREADS], s2[SCAN_THREADS];
  const int t = threadIdx.x;
  const int per = (B + SCAN_THREADS - 1) / SCAN_THREADS;
  const int lo = min(B, t * per), hi = min(B, lo + per);
  long long a = 0, b = 0;
  bool neg = false;
  for (int s = lo; s < hi; ++s) {
    long long n = len[s];
    neg |= n < 0;
    a += n;
    b += n * n;
  }
  s1[t] = a;
  s2[t] = b;
  __syncthreads();
  for (int off = 1; off < SCAN_THREADS; off <<= 1) {   // inclusive Hillis-Steele scan
    long long va = 0, vb = 0;
    if (t >= off) { va = s1[t - off]; vb = s2[t - off]; }
    __syncthreads();
    s1[t] += va;
    s2[t] += vb;
    __syncthreads();
  }
  long long ea = s1[t] - a, eb = s2[t] - b;            // exclusive prefix of this thread's chunk
  for (int s = lo; s < hi; ++s) {
    long long n = len[s];
    tok_off[s] = ea;
    pair_off[s] = eb;
    ea += n;
    eb += n * n;
  }
  if (t == SCAN_THREADS - 1) {
    tok_off[B] = s1[t];
    pair_off[B] = s2[t];
    if ((s1[t] != T1 || s2[t] != T2) && status) atomicCAS(status, 0, (int)NT_ERR_INCONSISTENT);
  }
  if (neg && status) atomicCAS(status, 0, (int)NT_ERR_INCONSISTENT);
}

__device__ inline int search_global(const int64_t* off, int B, long long p) {
  int lo = 0, hi = B;
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (off[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

__global__ void row_splits_kernel(const int64_t* __restrict__ len, const int64_t* __restrict__ tok_off,
                                  const int64_t* __restrict__ pair_off, int B, long long T1, long long T2,
                                  int64_t* __restrict__ row_splits) {
  if (tok_off[B] != T1 || pair_off[B] != T2) return;   // inconsistent totals: flagged by the scan
  long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t > T1) return;
  if (t == T1) { row_splits[t] = T2; return; }
  int s = search_global(tok_off, B, t);
  row_splits[t] = pair_off[s] + (t - tok_off[s]) * len[s];
}

constexpr int DEC_THREADS = 256;
constexpr int DEC_PER_THREAD = 4;
constexpr int DEC_SMEM_B = 2048;

__global__ void __launch_bounds__(DEC_THREADS)
decode_kernel(const int64_t* __restrict__ len, const int64_t* __restrict__ tok_off,
              const int64_t* __restrict__ pair_off, int B, long long T1, long long T2,
              int32_t* __restrict__ ps, int32_t* __restrict__ pi, int32_t* __restrict__ pj,
              int64_t* __restrict__ grow, int64_t* __restrict__ gcol) {
  if (tok_off[B] != T1 || pair_off[B] != T2) return;
  __shared__ long long so[DEC_SMEM_B + 1];
  const bool in_smem = B <= DEC_SMEM_B;
  if (in_smem) {
    for (int s = threadIdx.x; s <= B; s += DEC_THREADS) so[s] = pair_off[s];
    __syncthreads();
  }
  const long long base = (long long)blockIdx.x * (DEC_THREADS * DEC_PER_THREAD);
#pragma unroll
  for (int u = 0; u < DEC_PER_THREAD; ++u) {
    long long p = base + u * DEC_THREADS + threadIdx.x;
    if (p >= T2) return;
    int s;
    if (in_smem) {
      int lo = 0, hi = B;
      while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (so[mid] <= p) lo = mid; else hi = mid;
      }
      s = lo;
    } else {
      s = search_global(pair_off, B, p);
    }
    const long long o = in_smem ? so[s] : (long long)pair_off[s];
    const long long n = len[s];
    const unsigned long long r = (unsigned long long)(p - o);
    long long i, j;
    if (r <= 0xFFFFFFFFull && n <= 0xFFFFFFFFll) {
      unsigned int q = (unsigned int)r / (unsigned int)n;
      i = q;
      j = (long long)((unsigned int)r - q * (unsigned int)n);
    } else {
      i = (long long)(r / (unsigned long long)n);
      j = (long long)(r - (unsigned long long)i * (unsigned long long)n);
    }
    if (ps) {
      ps[p] = s;
      pi[p] = (int32_t)i;
      pj[p] = (int32_t)j;
    }
    if (grow) {
      const long long t0 = tok_off[s];
      grow[p] = t0 + i;
      gcol[p] = t0 + j;
    }
  }
}

}  // namespace ntp

using namespace ntp;

extern "C" nt_status nt_offsets_build(const int64_t* lengths_d, int32_t B, int64_t T1, int64_t T2,
                                      int64_t* tok_off_d, int64_t* pair_off_d, int64_t* row_splits_d,
                                      int32_t* pos_sample_d, int32_t* pos_i_d, int32_t* pos_j_d,
                                      int64_t* gather_rows_d, int64_t* gather_cols_d,
                                      int32_t* status_d, nt_stream stream_) {
  cudaStream_t stream = (cudaStream_t)stream_;
  if (B < 0 || T1 < 0 || T2 < 0) return NT_ERR_INVALID_ARG;
  if (!tok_off_d || !pair_off_d) return NT_ERR_INVALID_ARG;
  if (B > 0 && !lengths_d) return NT_ERR_INVALID_ARG;
  const bool want_pos = pos_sample_d || pos_i_d || pos_j_d;
  if (want_pos && !(pos_sample_d && pos_i_d && pos_j_d)) return NT_ERR_INVALID_ARG;
  const bool want_gather = gather_rows_d || gather_cols_d;
  if (want_gather && !(gather_rows_d && gather_cols_d)) return NT_ERR_INVALID_ARG;

  {
    LaunchScope ls("offsets_scan", stream);
    scan_lengths_kernel<<<1, SCAN_THREADS, 0, stream>>>(lengths_d, B, T1, T2, tok_off_d, pair_off_d, status_d);
  }
  if (row_splits_d) {
    long long n = T1 + 1;
    LaunchScope ls("offsets_row_splits", stream);
    row_splits_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(lengths_d, tok_off_d, pair_off_d, B, T1, T2,
                                                                      row_splits_d);
  }
  if ((want_pos || want_gather) && T2 > 0) {
    const long long per_block = DEC_THREADS * DEC_PER_THREAD;
    long long blocks = (T2 + per_block - 1) / per_block;
    if (blocks > 0x7FFFFFFFll) return NT_ERR_UNSUPPORTED;
    LaunchScope ls("offsets_decode", stream);
    decode_kernel<<<(unsigned)blocks, DEC_THREADS, 0, stream>>>(lengths_d, tok_off_d, pair_off_d, B, T1, T2,
                                                               pos_sample_d, pos_i_d, pos_j_d, gather_rows_d,
                                                               gather_cols_d);
  }
  return cuda_ok();
}
