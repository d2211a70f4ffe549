// Shape-generic CUDA-core kernels (any widths, float or bf16 storage, float arithmetic).
// They are the float path of the library and serve bf16 shapes that have no tensor-core kernel.
#pragma once
#include "common.cuh"

namespace ntp {

enum AMode { A_ROWMAJOR = 0, A_CHANNEL_MAJOR = 1 };
enum OutMode { O_STORE = 0, O_ACCUM = 1, O_CHANNEL_MAJOR = 2 };
enum Act { ACT_NONE = 0, ACT_SIGMOID = 1, ACT_SILU = 2 };   // with W2: gate activation (0 / 1: sigmoid, 2: SiLU)

// out = epilogue( prologue(A) W^T ) over the packed rows [row0, row0 + rows)
struct ProjArgs {
  const void* A;        // rows x K (row-major, ld = K) or channel-major pair layout with K channels
  int a_mode;
  long long row0, rows;
  int K;
  const void* gateA;    // nullable: row-major [.. , K] elementwise multiplier of A (same dtype)
  const void* ln_g;     // nullable: LayerNorm over K before the product
  const void* ln_b;
  float eps;
  const void* W1;       // [Nout, K]
  const void* W2;       // nullable: value = gate(A W1^T) * (A W2^T), gate = sigmoid unless act == ACT_SILU
  int Nout;
  int act;              // activation (W2 == NULL) or gate kind (W2 != NULL)
  void* out;
  int out_mode;         // O_STORE / O_ACCUM: row-major [.., Nout]; O_CHANNEL_MAJOR: pair layout, Nout channels
  const void* gateO;    // nullable: row-major [.., Nout]; value *= gateO before store/accumulate
  int out_f32;          // output buffer holds float regardless of the storage dtype
};

template <typename T>
nt_status launch_proj(const ProjArgs& a, const BatchMeta& m, cudaStream_t st, const char* name);

// t[c][i][j] = sum_k a[c][i][k] b[c][j][k] on channel-major buffers with C channels
template <typename T>
nt_status launch_contract(const T* a, const T* b, T* t, int C, const BatchMeta& m, cudaStream_t st, bool incoming = false);

// z[p,:] = LN(u[row(p)] + v[col(p)]) * gamma + beta;  u, v float [T1, c_z]
template <typename T>
nt_status launch_broadcast_ln(const float* u, const float* v, const T* gamma, const T* beta, float eps, int c_z,
                              T* z, const BatchMeta& m, cudaStream_t st, bool accumulate = false);

// softmax attention over attention rows.  pair order: rows are (s, i) and bias (nullable) is the
// head-major channel-major buffer; token order: one row per sample.
template <typename T>
nt_status launch_attn_core(const T* q, const T* k, const T* v, const T* bias, T* o, int H, int d, int pair_order,
                           const BatchMeta& m, cudaStream_t st, int skip_max_n = -1, float bias_scale = 1.0f);

template <typename T>
nt_status launch_segment_reduce(const T* v, T* out, const int64_t* splits, long long G, int C, int mean,
                                cudaStream_t st);

}  // namespace ntp
