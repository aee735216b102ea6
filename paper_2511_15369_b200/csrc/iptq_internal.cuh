// Argument structs and launcher prototypes shared by the translation units of the library (linear.cu,
// attention.cu, nonlinear.cu, block.cu): one definition, so that a field added on one side cannot go unnoticed
// on the other.
#pragma once

#include "iptq_common.cuh"

namespace iptq {

// ---------------------------------------------------------------- INT8 linear layer (linear.cu)
struct LinearArgs {
    const int8_t* x; const int8_t* w;                          // w already int8 [N, K]
    const int32_t* bias; const int32_t* mult; const int8_t* shift;
    int32_t out_zp;
    const int8_t* residual; const iptq_requant* residual_rq;
    const iptq_gelu_consts* gelu;                              // non-null: FC1 + GELU epilogue
    int8_t* y;
    int64_t M; int N, K;
    StatusBlock* status;
    int out_bits = 8;                                          // width of the output activations (plain and residual epilogues)
};
// Host-side argument checks of linear_launch() alone: nothing is enqueued.
int linear_check(const LinearArgs& a);
int linear_launch(const LinearArgs& a, cudaStream_t st);
int unpack_int4_launch(const void* packed, int8_t* out, int64_t n_elems, cudaStream_t st);
int unpack_int4_multi_launch(const void* const* packed, int8_t* const* out, const int64_t* n_elems, int count,
                             cudaStream_t st);

// ---------------------------------------------------------------- LayerNorm (nonlinear.cu)
int layernorm_launch(const int8_t* x, int8_t* y, int64_t rows, int dim, const int32_t* gq, const int32_t* bq,
                     const uint8_t* ptf, const iptq_ln_consts* consts, cudaStream_t st);

// ---------------------------------------------------------------- fused attention (attention.cu)
// Strided q/k/v so that the encoder block can read heads straight out of the fused QKV activation.
struct AttnArgs {
    const int8_t *q, *k, *v;
    int64_t tok_stride, head_stride, batch_stride;     // in bytes (= elements)
    int8_t* out;
    int64_t B; int H, N, dh;
    const int32_t* bias; const uint8_t* mask_id;
    const iptq_softmax_consts* sm; const iptq_requant* out_rq;
    StatusBlock* status;
    const int32_t* bias_t;  // N <= 64: the bias as iptq_attention_bias_prepare() lays it out (16-byte aligned), or null
};
int attention_launch(const AttnArgs& a, cudaStream_t st);

}  // namespace iptq
