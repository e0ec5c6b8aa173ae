// Tensor-core (tcgen05) backend: internal interface between the C-ABI layer and the pipelines.
#pragma once
#include "mw_common.cuh"
#include "mw_net.cuh"

namespace mw {

struct TcMapCache;
struct TcProgram;
// programs (whole phases in one launch) are rebuilt only when a buffer they name has moved
enum { MW_PROG_PHASE1 = 0, MW_PROG_PHASE2, MW_PROG_BP_FWD, MW_PROG_BP_BWD, MW_PROG_COUNT };
// variants of a program: which home of the Newton-Schulz iterate it starts from (0, 1), cold or
// refreshing (+2).  A training loop alternates between two of them; each is built once.
constexpr int kProgVariants = 4;
// 1: dense nets that qualify run the forward sweep as chained programs (mw_set_sweep_chains)
extern int g_sweep_chains;
struct TensorState {
  TcMapCache* cache = nullptr;
  TcProgram* prog[MW_PROG_COUNT][kProgVariants] = {};
  std::vector<const void*> key[MW_PROG_COUNT][kProgVariants];
  // the forward sweep as chained programs, one per run of layers that fits a product table
  // (two variants: the inverses' current home)
  std::vector<TcProgram*> sweep[2];
  std::vector<const void*> sweep_key[2];
  // LU-parameterised nets: the products that turn a chunk of layers' factors into W and W^-1
  // ([0]: W only, for the backprop reference; [1]: both), one program per chunk of layers
  std::vector<TcProgram*> lu_prog[2];
  std::vector<std::vector<const void*>> lu_key[2];
};

// convolutional nets on the tensor cores (mw_conv_pipeline.cu): stride-1 same-size convolutions
// with 64 channels, leaky-ReLU or no activation, MW_F32, optionally a linear head
bool conv_tensor_supported(const mw_net* n);
void conv_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start);
mw_status conv_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                      const void* target, void* g0, double* loss_out, void* ws,
                                      cudaStream_t s);
mw_status conv_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                    const void* g0, void* const* dW, void* ws, cudaStream_t s);
mw_status conv_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                               const void* target, void* const* dW, double* loss_out, void* ws,
                               cudaStream_t s);

// the fully submersive strided CNN (mw_sconv_pipeline.cu): stride-2 convolutions meeting Lemma 1
// with 64 or 128 channels, leaky-ReLU or no activation, MW_F32, loss on the last feature map
bool sconv_tensor_supported(const mw_net* n);
void sconv_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start);
mw_status sconv_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                       const void* target, void* g0, double* loss_out, void* ws,
                                       cudaStream_t s);
mw_status sconv_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                     const void* g0, void* const* dW, void* ws, cudaStream_t s);
mw_status sconv_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                                const void* target, void* const* dW, double* loss_out, void* ws,
                                cudaStream_t s);

// the 1-D CNN with fragmental checkpoints (mw_conv1d_pipeline.cu): k = 3, stride 1, padding 1
bool conv1d_tensor_supported(const mw_net* n);
void conv1d_tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start);
mw_status conv1d_tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                        const void* target, void* g0, double* loss_out, void* ws,
                                        cudaStream_t s);
mw_status conv1d_tensor_forward_sweep(mw_net* n, const void* const* params, const void* x,
                                      const void* g0, void* const* dW, void* ws, cudaStream_t s);
mw_status conv1d_tensor_backprop(mw_net* n, const void* const* params, const void* x,
                                 const void* target, void* const* dW, double* loss_out, void* ws,
                                 cudaStream_t s);

// true when every layer of the net has a tensor-core path (dense, sizes multiples of 64,
// MW_F32 or MW_BF16_F32ACC)
bool tensor_supported(const mw_net* n);
// appends the backend's transient regions to `lay` starting at byte `start`; sets lay.total
void tensor_layout(mw_net* n, bool backprop, Layout& lay, size_t start);
void tensor_destroy(mw_net* n);

mw_status tensor_input_cotangent(mw_net* n, const void* const* params, const void* x,
                                 const void* target, void* g0, double* loss_out, void* ws,
                                 cudaStream_t s);
mw_status tensor_forward_sweep(mw_net* n, const void* const* params, const void* x, const void* g0,
                               void* const* dW, void* ws, cudaStream_t s);
mw_status tensor_backprop(mw_net* n, const void* const* params, const void* x, const void* target,
                          void* const* dW, double* loss_out, void* ws, cudaStream_t s);

}  // namespace mw
