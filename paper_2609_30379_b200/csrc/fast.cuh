// bf16 kernels tuned for sm_100a.  Memory-bound steps stay on CUDA cores with 16-byte vector
// access; dense contractions use tcgen05 tensor-core tiles with TMEM accumulators.
#pragma once
#include "common.cuh"

namespace ntp {

bool fast_broadcast_supported(int c_z);
nt_status fast_broadcast_ln(const float* u, const float* v, const void* gamma, const void* beta, float eps, int c_z,
                            void* z, const BatchMeta& m, cudaStream_t st);

bool fast_segment_reduce_supported(int C);
nt_status fast_segment_reduce(const void* v, void* out, const int64_t* splits, long long G, int C, int mean,
                              cudaStream_t st);

// attention core on tensor cores (bf16, d in {16, 32, 64}); q, k, v, o row-major [rows, H*d], bias
// head-major channel-major (nullable)
bool fast_attn_core_supported(int H, int d);
nt_status fast_attn_core(const void* q, const void* k, const void* v, const void* bias, void* o, int H, int d,
                         int pair_order, const BatchMeta& m, cudaStream_t st);

// triangle contraction on tcgen05: a, b, t are three equally spaced channel-major buffers
// (b = a + stride, t = a + 2 * stride)
bool fast_contract_supported(int C);
nt_status fast_contract(const void* a, size_t buf_stride_bytes, int C, const BatchMeta& m, int* status,
                        cudaStream_t st);

// triangle input projection on tcgen05 (LayerNorm folded into the weights); `prep` is scratch of
// fast_tri_in_prep_bytes() for the folded weights
bool fast_tri_in_supported(int c_z, int c_h);
size_t fast_tri_in_prep_bytes(int c_z, int c_h);
nt_status fast_tri_in(const void* z, const nt_trimul_weights* W, float eps, int c_z, int c_h, void* a, void* b,
                      void* prep, const BatchMeta& m, int* status, cudaStream_t st);
nt_status fast_ln_fold_prep(const void* const* srcs, const int* rows, int nsrc, int K, const void* gamma,
                            const void* beta, void* out, void* c01, cudaStream_t st);

// attention input projection on tcgen05: q, k, v row-major, bias head-major (nullable)
bool fast_attn_in_supported(int c, int H, int d);
nt_status fast_attn_in(const void* z, const nt_attn_weights* W, float eps, int c, int H, int d, void* q, void* k,
                       void* v, void* bias, void* prep, const BatchMeta& m, int* status, cudaStream_t st);

// attention output stage on tcgen05, in place on z: z += (sigmoid(LN(z) W_g^T) * o) W_o^T
bool fast_attn_out_supported(int c, int H, int d);
nt_status fast_attn_out(void* z, const void* o, const nt_attn_weights* W, float eps, int c, int H, int d, void* prep,
                        const BatchMeta& m, int* status, cudaStream_t st);

// triangle output stage on tcgen05, in place on z: z += sigmoid(LN_in(z) W_g^T) * (LN_out(t) W_o^T)
bool fast_tri_out_supported(int c_z, int c_h);
size_t fast_tri_out_prep_bytes(int c_z, int c_h);
nt_status fast_tri_out(void* z, const void* t, const nt_trimul_weights* W, float eps, int c_z, int c_h, void* prep,
                       const BatchMeta& m, int* status, cudaStream_t st);

}  // namespace ntp
