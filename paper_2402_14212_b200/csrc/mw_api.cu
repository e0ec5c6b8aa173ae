// C-ABI entry points of the Moonwalk library: network description, workspace layout, and the
// CUDA-core (exact arithmetic) pipelines of the three calls.  The tensor-core pipelines live in
// mw_tensor_pipeline.cu and are selected per net (backend).
#include <cstring>
#include <new>

#include "mw_common.cuh"
#include "mw_conv.cuh"
#include "mw_net.cuh"
#include "mw_tc_gemm.cuh"
#include "mw_tensor.cuh"

using namespace mw;

long long mw::g_launch_count = 0;

// ---------------------------------------------------------------------------------------
// description and layout
// ---------------------------------------------------------------------------------------
namespace {

struct Bump {
  size_t cur = 0;
  Region take(size_t bytes) {
    Region r;
    r.off = cur;
    r.bytes = bytes;
    cur = align_up(cur + bytes, 256);
    return r;
  }
};

bool valid_layer(const mw_layer_desc& d, int idx, int L) {
  if (d.act < MW_ACT_NONE || d.act > MW_ACT_RELU) return false;
  // a leaky-ReLU of slope 0 is a ReLU: not submersive, its vijp would divide by zero
  if (d.act == MW_ACT_LEAKY_RELU && !(d.slope != 0.0 && d.slope - d.slope == 0.0)) return false;
  if (d.kind == MW_DENSE) return d.n_in > 0 && d.n_in == d.n_out;
  if (d.kind == MW_HEAD_LINEAR) return idx == L - 1 && d.n_in > 0 && d.n_out > 0 && d.act == MW_ACT_NONE;
  if (d.kind == MW_CONV1D)
    return d.H == 1 && d.W > 0 && d.C_in > 0 && d.C_in == d.C_out && d.k >= 2 && d.stride == 1 && d.pad == 1 &&
           d.k == 3;
  if (d.kind == MW_CONV2D) {
    if (!(d.H > 0 && d.W > 0 && d.C_in > 0 && d.C_in == d.C_out && d.k >= 1 && d.pad >= 0 && d.stride >= 1))
      return false;
    // same-size stride-1 layers (vijp by iteration on the centre tap), or Lemma 1 (i)
    if (d.stride == 1) return d.k == 2 * d.pad + 1;
    if (!(d.k > d.pad && d.stride > d.pad && d.H + 2 * d.pad >= d.k && d.W + 2 * d.pad >= d.k)) return false;
    const int Ho = (d.H + 2 * d.pad - d.k) / d.stride + 1, Wo = (d.W + 2 * d.pad - d.k) / d.stride + 1;
    return d.H > d.stride * (Ho - 1) && d.W > d.stride * (Wo - 1);
  }
  return false;
}

void build_layout(mw_net* n, bool backprop, Layout& lay) {
  Bump b;
  const size_t es = n->es;
  const int L = n->L;
  lay = Layout();
  lay.status = b.take(256);
  lay.partials = b.take(sizeof(double) * 1024 + sizeof(double) * (size_t)n->B);
  lay.mask.resize(L);
  lay.frag_cnt.resize(L);
  lay.frag_off.resize(L);
  lay.frag_rank.resize(L);
  lay.frag_vals.resize(L);
  lay.reseed.resize(L + 1);
  lay.stored_act.resize(L + 1);
  lay.inv.resize(L);
  lay.w_planes.resize(L);
  int64_t max_elems = 0, max_w = 0, max_inv = 0;
  for (int l = 0; l < L; ++l) {
    const LayerInfo& li = n->info[l];
    if (li.in_elems > max_elems) max_elems = li.in_elems;
    if (li.out_elems > max_elems) max_elems = li.out_elems;
    if (li.w_elems > max_w) max_w = li.w_elems;
    const int64_t inv_e = n->layers[l].kind == MW_CONV2D
                              ? (int64_t)li.inv_n * li.inv_n + li.w_elems
                              : (int64_t)li.inv_n * li.inv_n;
    if (inv_e > max_inv) max_inv = inv_e;
  }
  // ---- residual stores (survive between phases) ----
  for (int l = 0; l < L; ++l) lay.mask[l] = b.take(sizeof(uint32_t) * n->info[l].rows * n->info[l].wpr);
  if (!backprop) {
    lay.frag_total = b.take(sizeof(uint32_t) * (size_t)(L + 1));
    for (int l = 0; l < L; ++l) {
      if (n->layers[l].act == MW_ACT_RELU) {
        lay.frag_cnt[l] = b.take(sizeof(uint32_t) * n->info[l].rows);
        lay.frag_off[l] = b.take(sizeof(uint32_t) * n->info[l].rows);
        if (n->backend == MW_BACKEND_TENSOR)
          lay.frag_rank[l] = b.take(sizeof(uint32_t) * n->info[l].rows * ((n->info[l].cols + 63) / 64));
        lay.frag_vals[l] = b.take((n->opts.prec == MW_F64 ? 8 : 4) * (size_t)n->info[l].out_elems);
      }
    }
    for (int l = 1; l < L; ++l)
      if (is_reseed(n, l)) {
        // dense tensor-core nets keep the checkpoint as bf16 term planes (3 for MW_F32, 2 otherwise)
        size_t per = n->opts.prec == MW_F64 ? 8 : 4;
        if (n->backend == MW_BACKEND_TENSOR && n->layers[0].kind == MW_DENSE && n->opts.prec == MW_F32) per = 6;
        lay.reseed[l] = b.take(per * (size_t)n->info[l - 1].out_elems);
      }
    if (n->layers[L - 1].kind == MW_HEAD_LINEAR)
      lay.h_last = b.take((n->opts.prec == MW_F64 ? 8 : 4) * (size_t)n->info[L - 1].out_elems);
  } else {
    const size_t aes = n->opts.prec == MW_F64 ? 8 : (n->opts.prec == MW_F32 ? 4 : 2);
    const int planes = (n->backend == MW_BACKEND_TENSOR && n->opts.prec == MW_F32) ? 3 : 1;
    const size_t per = (n->backend == MW_BACKEND_TENSOR) ? 2 * (size_t)planes : aes;
    for (int l = 1; l < L; ++l) lay.stored_act[l] = b.take(per * (size_t)n->info[l - 1].out_elems);
  }
  lay.residual = b.cur;
  // ---- transient buffers ----
  if (n->backend == MW_BACKEND_SIMT) {
    for (int i = 0; i < 2; ++i) lay.act[i] = b.take(es * max_elems);
    for (int i = 0; i < 2; ++i) lay.cot[i] = b.take(es * max_elems);
    lay.z = b.take(es * max_elems);
    lay.gz = b.take(es * max_elems);
    bool any_conv = false;
    size_t wgrad_part = 0;
    for (int l = 0; l < L; ++l)
      if (n->layers[l].kind == MW_CONV2D) {
        any_conv = true;
        size_t p = es * (size_t)conv_wgrad_slices(n->info[l].rows) * n->info[l].w_elems;
        if (p > wgrad_part) wgrad_part = p;
      }
    if (any_conv) {
      lay.aux0 = b.take(es * max_elems > wgrad_part ? es * max_elems : wgrad_part);
      lay.aux1 = b.take(es * max_elems);
    }
    if (!backprop) {
      if (n->opts.resident_inverse) {
        for (int l = 0; l < L; ++l) {
          const LayerInfo& li = n->info[l];
          const int64_t e = n->layers[l].kind == MW_CONV2D ? (int64_t)li.inv_n * li.inv_n + li.w_elems
                                                          : (int64_t)li.inv_n * li.inv_n;
          lay.inv[l] = b.take(es * (size_t)e);
        }
      } else {
        Region slot = b.take(es * (size_t)max_inv);
        for (int l = 0; l < L; ++l) lay.inv[l] = slot;
      }
      int max_n = 0;
      for (int l = 0; l < L; ++l)
        if (n->info[l].inv_n > max_n) max_n = n->info[l].inv_n;
      lay.inv_scratch = b.take(es * 2 * (size_t)max_n * max_n + 64);
    }
  } else {
    tensor_layout(n, backprop, lay, b.cur);
    b.cur = lay.total;
  }
  lay.total = b.cur;
}

}  // namespace

extern "C" mw_status mw_net_create(const mw_layer_desc* layers, int32_t n_layers, int32_t batch,
                                   const mw_net_opts* opts, mw_net** out) {
  if (!layers || !opts || !out || n_layers < 1 || batch < 1) return MW_ERR_INVALID_ARG;
  if (opts->prec < MW_F64 || opts->prec > MW_BF16_F32ACC) return MW_ERR_INVALID_ARG;
  if (opts->loss < MW_LOSS_HALF_SSE || opts->loss > MW_LOSS_XENT_MEAN) return MW_ERR_INVALID_ARG;
  if (opts->reseed_every < 0 || opts->conv_vijp_iters < 0 || opts->inverse_iters < 0 || opts->frag_block < 0)
    return MW_ERR_INVALID_ARG;
  if (opts->backend < MW_BACKEND_AUTO || opts->backend > MW_BACKEND_TENSOR) return MW_ERR_INVALID_ARG;
  if (opts->warm_inverse != 0 && opts->warm_inverse != 1) return MW_ERR_INVALID_ARG;
  if (opts->lu_param != 0 && opts->lu_param != 1) return MW_ERR_INVALID_ARG;
  if (opts->lu_param) {
    // triangular factors as parameters: dense nets on the tensor cores in MW_F32, inverses resident
    if (opts->prec != MW_F32 || opts->backend == MW_BACKEND_SIMT || !opts->resident_inverse || opts->warm_inverse)
      return MW_ERR_UNSUPPORTED;
    for (int l = 0; l < n_layers; ++l)
      if (layers[l].kind != MW_DENSE || layers[l].n_in % 128 != 0) return MW_ERR_UNSUPPORTED;
  }
  for (int l = 0; l < n_layers; ++l) {
    if (layers[l].kind < MW_DENSE || layers[l].kind > MW_CONV1D) return MW_ERR_INVALID_ARG;
    if (!valid_layer(layers[l], l, n_layers)) return MW_ERR_UNSUPPORTED;
  }
  mw_net* n = new (std::nothrow) mw_net();
  if (!n) return MW_ERR_INVALID_ARG;
  n->layers.assign(layers, layers + n_layers);
  n->L = n_layers;
  n->B = batch;
  n->opts = *opts;
  n->es = opts->prec == MW_F64 ? 8 : 4;
  n->info.resize(n_layers);
  int64_t prev_out = -1;
  for (int l = 0; l < n_layers; ++l) {
    const mw_layer_desc& d = n->layers[l];
    LayerInfo& li = n->info[l];
    if (d.kind == MW_CONV1D) {
      li.rows = (int64_t)batch * d.W;
      li.cols = d.C_out;
      li.in_elems = li.rows * d.C_in;
      li.out_elems = li.rows * d.C_out;
      li.w_elems = (int64_t)d.k * d.C_in * d.C_out;
      li.inv_n = d.C_in;
    } else if (d.kind == MW_CONV2D) {
      const int Ho = (d.H + 2 * d.pad - d.k) / d.stride + 1, Wo = (d.W + 2 * d.pad - d.k) / d.stride + 1;
      li.rows = (int64_t)batch * Ho * Wo;
      li.cols = d.C_out;
      li.in_elems = (int64_t)batch * d.H * d.W * d.C_in;
      li.out_elems = li.rows * d.C_out;
      li.w_elems = (int64_t)d.k * d.k * d.C_in * d.C_out;
      li.inv_n = d.C_in;
    } else {
      li.rows = batch;
      li.cols = d.n_out;
      li.in_elems = (int64_t)batch * d.n_in;
      li.out_elems = (int64_t)batch * d.n_out;
      li.w_elems = (int64_t)d.n_in * d.n_out;
      li.inv_n = d.kind == MW_DENSE ? d.n_in : 0;
    }
    li.wpr = (li.cols + 31) / 32;
    if (prev_out >= 0 && prev_out != li.in_elems) {
      delete n;
      return MW_ERR_INVALID_ARG;
    }
    prev_out = li.out_elems;
  }
  if (opts->loss == MW_LOSS_XENT_MEAN && n->layers[n_layers - 1].kind != MW_HEAD_LINEAR &&
      n->layers[n_layers - 1].kind != MW_DENSE) {
    delete n;
    return MW_ERR_UNSUPPORTED;
  }
  // backend
  const bool tensor_ok = tensor_supported(n);
  if (opts->backend == MW_BACKEND_TENSOR && !tensor_ok) {
    delete n;
    return MW_ERR_UNSUPPORTED;
  }
  if (opts->backend == MW_BACKEND_AUTO) n->backend = tensor_ok ? MW_BACKEND_TENSOR : MW_BACKEND_SIMT;
  else n->backend = opts->backend;
  if (opts->lu_param && n->backend != MW_BACKEND_TENSOR) {
    delete n;
    return MW_ERR_UNSUPPORTED;
  }
  if (n->backend == MW_BACKEND_SIMT && opts->prec == MW_BF16_F32ACC) {
    delete n;
    return MW_ERR_UNSUPPORTED;
  }
  // strided and 1-D convolutions only have the tensor-core path; a conv net is all of one kind
  for (int l = 0; l < n_layers; ++l) {
    const mw_layer_desc& d = n->layers[l];
    if ((d.kind == MW_CONV1D || n->layers[0].kind == MW_CONV1D) &&
        (d.kind != n->layers[0].kind || n->backend != MW_BACKEND_TENSOR)) {
      delete n;
      return MW_ERR_UNSUPPORTED;
    }
    if (d.kind == MW_CONV2D && (d.stride != n->layers[0].stride || n->layers[0].kind != MW_CONV2D ||
                                (d.stride != 1 && n->backend != MW_BACKEND_TENSOR))) {
      delete n;
      return MW_ERR_UNSUPPORTED;
    }
  }
  build_layout(n, false, n->mwl);
  build_layout(n, true, n->bpl);
  n->lean_seed = n->backend == MW_BACKEND_TENSOR && n->layers[0].kind == MW_CONV2D && n->layers[0].stride != 1;
  *out = n;
  return MW_OK;
}

extern "C" void mw_net_destroy(mw_net* net) {
  if (!net) return;
  tensor_destroy(net);
  delete net;
}

extern "C" mw_status mw_workspace_bytes(const mw_net* net, size_t* moonwalk_bytes,
                                        size_t* backprop_bytes, size_t residual_bytes[2]) {
  if (!net) return MW_ERR_INVALID_ARG;
  if (moonwalk_bytes) *moonwalk_bytes = net->mwl.total;
  if (backprop_bytes) *backprop_bytes = net->bpl.total;
  if (residual_bytes) {
    residual_bytes[0] = net->mwl.residual;
    residual_bytes[1] = net->bpl.residual;
  }
  return MW_OK;
}

extern "C" const char* mw_status_string(mw_status s) {
  switch (s) {
    case MW_OK: return "ok";
    case MW_ERR_INVALID_ARG: return "invalid argument";
    case MW_ERR_UNSUPPORTED: return "unsupported layer or size";
    case MW_ERR_WORKSPACE: return "workspace null, misaligned or too small";
    case MW_ERR_STATE: return "forward sweep without a matching input-cotangent pass";
    case MW_ERR_NOT_SUBMERSIVE: return "layer Jacobian could not be inverted to tolerance";
    case MW_ERR_TIMEOUT: return "bounded device-side wait expired";
    case MW_ERR_CUDA: return "CUDA call failed";
  }
  return "unknown status";
}

// ---------------------------------------------------------------------------------------
// CUDA-core pipelines
// ---------------------------------------------------------------------------------------
namespace {

mw_status check_ws(const void* ws, size_t bytes, size_t need) {
  if (!ws || ((uintptr_t)ws & 255u) != 0 || bytes < need) return MW_ERR_WORKSPACE;
  return MW_OK;
}

template <typename T>
mw_status lin_forward(const mw_net* n, int l, const T* W, const T* x, T* z, cudaStream_t s) {
  const mw_layer_desc& d = n->layers[l];
  if (d.kind == MW_CONV2D)
    return conv_igemm<T>(x, W, z, nullptr, n->B, d.H, d.W, d.C_in, d.C_out, d.k, d.pad, +1, 0, 0, s);
  return gemm_simt<T>(0, 1, n->B, d.n_out, d.n_in, 1.0, x, d.n_in, W, d.n_in, 0.0, z, d.n_out, s);
}

template <typename T>
mw_status lin_vjp_input(const mw_net* n, int l, const T* W, const T* gz, T* h, cudaStream_t s) {
  const mw_layer_desc& d = n->layers[l];
  if (d.kind == MW_CONV2D)
    return conv_igemm<T>(gz, W, h, nullptr, n->B, d.H, d.W, d.C_out, d.C_in, d.k, d.pad, -1, 1, 0, s);
  return gemm_simt<T>(0, 0, n->B, d.n_in, d.n_out, 1.0, gz, d.n_out, W, d.n_in, 0.0, h, d.n_in, s);
}

template <typename T>
mw_status lin_wgrad(const mw_net* n, int l, const T* x, const T* gz, T* dW, void* ws,
                    const Layout& lay, cudaStream_t s) {
  const mw_layer_desc& d = n->layers[l];
  if (d.kind == MW_CONV2D)
    return conv_wgrad<T>(x, gz, dW, at<T>(ws, lay.aux0), n->B, d.H, d.W, d.C_in, d.C_out, d.k, d.pad, s);
  return gemm_simt<T>(1, 0, d.n_out, d.n_in, n->B, 1.0, gz, d.n_out, x, d.n_in, 0.0, dW, d.n_in, s);
}

// W^-1 (dense) or centre-tap inverse + folded kernel (conv) into the layer's inverse region
template <typename T>
mw_status prep_inverse(const mw_net* n, int l, const T* W, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  const mw_layer_desc& d = n->layers[l];
  DeviceStatus* st = status_of(ws, lay);
  T* inv = at<T>(ws, lay.inv[l]);
  T* scratch = at<T>(ws, lay.inv_scratch);
  const double tol = sizeof(T) == 8 ? 1e-9 : 2e-4;
  if (d.kind == MW_HEAD_LINEAR) return MW_OK;
  const int m = n->info[l].inv_n;
  const T* block = W;
  if (d.kind == MW_CONV2D) block = W + (size_t)(d.pad * d.k + d.pad) * d.C_in * d.C_out;
  if (m <= 64) {
    MW_TRY(inverse_small<T>(block, m, inv, st, l, s));
  } else {
    int iters = n->opts.inverse_iters ? n->opts.inverse_iters : (sizeof(T) == 8 ? 8 : 6);
    MW_TRY(inverse_newton_simt<T>(block, m, iters, inv, scratch, st, l, tol, s));
  }
  if (d.kind == MW_CONV2D) {
    // w^[tap] = W_c^-1 w[tap] for tap != centre, zero at the centre
    T* what = inv + (size_t)m * m;
    const size_t tap_e = (size_t)d.C_in * d.C_out;
    for (int tap = 0; tap < d.k * d.k; ++tap) {
      if (tap == d.pad * d.k + d.pad) {
        MW_TRY(zero_array<T>(what + tap * tap_e, (int64_t)tap_e, s));
      } else {
        MW_TRY(gemm_simt<T>(0, 0, m, d.C_out, m, 1.0, inv, m, W + tap * tap_e, d.C_out, 0.0,
                            what + tap * tap_e, d.C_out, s));
      }
    }
  }
  return MW_OK;
}

// g_z = vijp of the linear part: dense g_z = h W^-1; conv: fixed-point iteration
template <typename T>
mw_status lin_vijp(const mw_net* n, int l, const T* h, T* gz, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  const mw_layer_desc& d = n->layers[l];
  const T* inv = at<T>(ws, lay.inv[l]);
  if (d.kind == MW_DENSE)
    return gemm_simt<T>(0, 0, n->B, d.n_out, d.n_in, 1.0, h, d.n_in, inv, d.n_out, 0.0, gz, d.n_out, s);
  // conv
  const int C = d.C_in;
  const int64_t rows = n->info[l].rows;
  T* hp = at<T>(ws, lay.aux1);               // h' = h W_c^-T
  T* g2 = at<T>(ws, lay.aux0);
  const T* what = inv + (size_t)C * C;
  MW_TRY(gemm_simt<T>(0, 1, (int)rows, C, C, 1.0, h, C, inv, C, 0.0, hp, C, s));
  const int iters = n->opts.conv_vijp_iters;
  T* cur = gz;
  T* nxt = g2;
  if (iters % 2 == 1) { cur = g2; nxt = gz; }     // so that the last update lands in gz
  MW_CUDA_OK(cudaMemcpyAsync(cur, hp, sizeof(T) * rows * C, cudaMemcpyDeviceToDevice, s));
  for (int it = 0; it < iters; ++it) {
    MW_TRY(conv_igemm<T>(cur, what, nxt, hp, n->B, d.H, d.W, C, C, d.k, d.pad, -1, 1, 1, s));
    T* t = cur; cur = nxt; nxt = t;
  }
  return MW_OK;
}

template <typename T>
mw_status simt_forward_pass(mw_net* n, const Layout& lay, const void* const* params, const T* x,
                            void* ws, bool store_acts, T** y_out, cudaStream_t s) {
  // Phase I (or backprop's forward): returns the network output in *y_out
  const T* cur = x;
  for (int l = 0; l < n->L; ++l) {
    const LayerInfo& li = n->info[l];
    const mw_layer_desc& d = n->layers[l];
    T* z = at<T>(ws, lay.z);
    MW_TRY(lin_forward<T>(n, l, (const T*)params[l], cur, z, s));
    T* nxt = (store_acts && l + 1 < n->L) ? at<T>(ws, lay.stored_act[l + 1]) : at<T>(ws, lay.act[l & 1]);
    MW_TRY((act_forward_pack<T, T>(z, li.rows, li.cols, d.act, d.slope, nxt,
                                   at<uint32_t>(ws, lay.mask[l]), true, s)));
    cur = nxt;
  }
  *y_out = const_cast<T*>(cur);
  return MW_OK;
}

template <typename T>
mw_status simt_input_cotangent(mw_net* n, const void* const* params, const T* x, const void* target,
                               T* g0, double* loss_out, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  const int L = n->L;
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  if (n->opts.resident_inverse)
    for (int l = 0; l < L; ++l) MW_TRY(prep_inverse<T>(n, l, (const T*)params[l], ws, s));
  T* y = nullptr;
  MW_TRY(simt_forward_pass<T>(n, lay, params, x, ws, false, &y, s));
  T* h = at<T>(ws, lay.cot[0]);
  const LayerInfo& last = n->info[L - 1];
  MW_TRY(loss_cotangent<T>(y, target, last.rows, last.cols, n->opts.loss, h,
                           at<double>(ws, lay.partials), loss_out, s));
  if (n->layers[L - 1].kind == MW_HEAD_LINEAR)
    MW_CUDA_OK(cudaMemcpyAsync(at<T>(ws, lay.h_last), h, sizeof(T) * last.out_elems,
                               cudaMemcpyDeviceToDevice, s));
  int hi = 0;
  for (int l = L - 1; l >= 0; --l) {
    const LayerInfo& li = n->info[l];
    const mw_layer_desc& d = n->layers[l];
    const uint32_t* words = at<uint32_t>(ws, lay.mask[l]);
    if (d.act == MW_ACT_RELU) {
      MW_TRY(fragment_offsets(words, li.rows, li.cols, at<uint32_t>(ws, lay.frag_cnt[l]),
                              at<uint32_t>(ws, lay.frag_off[l]),
                              at<uint32_t>(ws, lay.frag_total) + l, nullptr, 0, s));
      MW_TRY(fragment_compact<T>(h, words, li.rows, li.cols, at<uint32_t>(ws, lay.frag_off[l]),
                                 at<T>(ws, lay.frag_vals[l]), s));
    }
    if (is_reseed(n, l + 1))
      MW_CUDA_OK(cudaMemcpyAsync(at<T>(ws, lay.reseed[l + 1]), h, sizeof(T) * li.out_elems,
                                 cudaMemcpyDeviceToDevice, s));
    const T* gz = h;
    if (d.act != MW_ACT_NONE) {
      T* g = at<T>(ws, lay.gz);
      MW_TRY(scale_by_mask<T>(h, words, li.rows, li.cols, d.act, d.slope, g, s));
      gz = g;
    }
    T* hprev = l == 0 ? g0 : at<T>(ws, lay.cot[hi ^ 1]);
    MW_TRY(lin_vjp_input<T>(n, l, (const T*)params[l], gz, hprev, s));
    h = hprev;
    hi ^= 1;
  }
  return MW_OK;
}

template <typename T>
mw_status simt_forward_sweep(mw_net* n, const void* const* params, const T* x, const T* g0,
                             void* const* dW, void* ws, cudaStream_t s) {
  const Layout& lay = n->mwl;
  const int L = n->L;
  const T* xc = x;
  const T* h = g0;
  for (int l = 0; l < L; ++l) {
    const LayerInfo& li = n->info[l];
    const mw_layer_desc& d = n->layers[l];
    const uint32_t* words = at<uint32_t>(ws, lay.mask[l]);
    if (!n->opts.resident_inverse) MW_TRY(prep_inverse<T>(n, l, (const T*)params[l], ws, s));
    T* z = at<T>(ws, lay.z);
    MW_TRY(lin_forward<T>(n, l, (const T*)params[l], xc, z, s));          // recompute
    T* gz = at<T>(ws, lay.gz);
    T* hn = at<T>(ws, lay.cot[l & 1]);
    const T* gz_used = gz;
    if (d.kind == MW_HEAD_LINEAR) {
      gz_used = at<T>(ws, lay.h_last);
    } else {
      MW_TRY(lin_vijp<T>(n, l, h, gz, ws, s));                            // vijp, linear part
      MW_TRY(activation_vijp<T>(gz, words, li.rows, li.cols, d.act, d.slope,
                                d.act == MW_ACT_RELU ? at<uint32_t>(ws, lay.frag_off[l]) : nullptr,
                                d.act == MW_ACT_RELU ? at<T>(ws, lay.frag_vals[l]) : nullptr, hn,
                                d.act == MW_ACT_RELU ? gz : nullptr, s)); // vijp, activation part
    }
    if (dW[l]) MW_TRY(lin_wgrad<T>(n, l, xc, gz_used, (T*)dW[l], ws, lay, s));  // g_i
    if (l + 1 < L) {
      T* xn = at<T>(ws, lay.act[l & 1]);
      MW_TRY((act_forward_pack<T, T>(z, li.rows, li.cols, d.act, d.slope, xn,
                                     const_cast<uint32_t*>(words), false, s)));
      xc = xn;
      h = is_reseed(n, l + 1) ? at<T>(ws, lay.reseed[l + 1]) : hn;
    }
  }
  return MW_OK;
}

template <typename T>
mw_status simt_backprop(mw_net* n, const void* const* params, const T* x, const void* target,
                        void* const* dW, double* loss_out, void* ws, cudaStream_t s) {
  const Layout& lay = n->bpl;
  const int L = n->L;
  MW_CUDA_OK(cudaMemsetAsync(at<char>(ws, lay.status), 0, 256, s));
  T* y = nullptr;
  MW_TRY(simt_forward_pass<T>(n, lay, params, x, ws, true, &y, s));
  T* h = at<T>(ws, lay.cot[0]);
  const LayerInfo& last = n->info[L - 1];
  MW_TRY(loss_cotangent<T>(y, target, last.rows, last.cols, n->opts.loss, h,
                           at<double>(ws, lay.partials), loss_out, s));
  int hi = 0;
  for (int l = L - 1; l >= 0; --l) {
    const LayerInfo& li = n->info[l];
    const mw_layer_desc& d = n->layers[l];
    const uint32_t* words = at<uint32_t>(ws, lay.mask[l]);
    const T* gz = h;
    if (d.act != MW_ACT_NONE) {
      T* g = at<T>(ws, lay.gz);
      MW_TRY(scale_by_mask<T>(h, words, li.rows, li.cols, d.act, d.slope, g, s));
      gz = g;
    }
    const T* xin = l == 0 ? x : at<T>(ws, lay.stored_act[l]);
    if (dW[l]) MW_TRY(lin_wgrad<T>(n, l, xin, gz, (T*)dW[l], ws, lay, s));
    if (l > 0) {
      T* hprev = at<T>(ws, lay.cot[hi ^ 1]);
      MW_TRY(lin_vjp_input<T>(n, l, (const T*)params[l], gz, hprev, s));
      h = hprev;
      hi ^= 1;
    }
  }
  return MW_OK;
}

}  // namespace

extern "C" mw_status mw_input_cotangent(mw_net* net, const void* const* params, const void* x,
                                        const void* loss_target, void* g0_out, double* loss_out,
                                        void* workspace, size_t workspace_bytes, void* stream) {
  if (!net || !params || !x || !loss_target) return MW_ERR_INVALID_ARG;
  if (!g0_out && !net->lean_seed) return MW_ERR_INVALID_ARG;
  for (int l = 0; l < net->L; ++l)
    if (!params[l]) return MW_ERR_INVALID_ARG;
  MW_TRY(check_ws(workspace, workspace_bytes, net->mwl.total));
  cudaStream_t s = (cudaStream_t)stream;
  net->ws_done = nullptr;
  mw_status r;
  if (net->backend == MW_BACKEND_TENSOR)
    r = tensor_input_cotangent(net, params, x, loss_target, g0_out, loss_out, workspace, s);
  else if (net->opts.prec == MW_F64)
    r = simt_input_cotangent<double>(net, params, (const double*)x, loss_target, (double*)g0_out,
                                     loss_out, workspace, s);
  else
    r = simt_input_cotangent<float>(net, params, (const float*)x, loss_target, (float*)g0_out,
                                    loss_out, workspace, s);
  if (r == MW_OK) {
    net->ws_done = workspace;
    net->x_done = x;
  }
  return r;
}

extern "C" mw_status mw_forward_sweep(mw_net* net, const void* const* params, const void* x,
                                      const void* g0, void* const* dW_out, void* workspace,
                                      size_t workspace_bytes, void* stream) {
  if (!net || !params || !x || !dW_out) return MW_ERR_INVALID_ARG;
  if (!g0 && !net->lean_seed) return MW_ERR_INVALID_ARG;
  for (int l = 0; l < net->L; ++l)
    if (!params[l]) return MW_ERR_INVALID_ARG;
  MW_TRY(check_ws(workspace, workspace_bytes, net->mwl.total));
  if (net->ws_done != workspace || net->x_done != x) return MW_ERR_STATE;
  cudaStream_t s = (cudaStream_t)stream;
  net->buckets_recorded = 0;
  mw_status r;
  if (net->backend == MW_BACKEND_TENSOR)
    r = tensor_forward_sweep(net, params, x, g0, dW_out, workspace, s);
  else if (net->opts.prec == MW_F64)
    r = simt_forward_sweep<double>(net, params, (const double*)x, (const double*)g0, dW_out, workspace, s);
  else
    r = simt_forward_sweep<float>(net, params, (const float*)x, (const float*)g0, dW_out, workspace, s);
  // buckets that the pipeline did not signal on its way are complete now at the latest
  if (r == MW_OK) record_buckets(net, net->L, s);
  return r;
}

extern "C" mw_status mw_sweep_bucket_events(mw_net* net, int32_t layers_per_bucket, void* const* events,
                                            int32_t n_events) {
  if (!net || layers_per_bucket < 0 || n_events < 0) return MW_ERR_INVALID_ARG;
  net->bucket_events.clear();
  net->bucket_layers = 0;
  if (layers_per_bucket == 0 || n_events == 0) return MW_OK;
  if (!events || n_events != (net->L + layers_per_bucket - 1) / layers_per_bucket) return MW_ERR_INVALID_ARG;
  for (int i = 0; i < n_events; ++i) {
    if (!events[i]) { net->bucket_events.clear(); return MW_ERR_INVALID_ARG; }
    net->bucket_events.push_back((cudaEvent_t)events[i]);
  }
  net->bucket_layers = layers_per_bucket;
  return MW_OK;
}

extern "C" mw_status mw_forward_sweep_apply(mw_net* net, const void* const* params, const void* x,
                                            const void* g0, double lr, void* const* params_out,
                                            void* workspace, size_t workspace_bytes, void* stream) {
  if (!net || !params || !params_out) return MW_ERR_INVALID_ARG;
  if (net->backend != MW_BACKEND_TENSOR || net->opts.prec != MW_F32 || net->opts.lu_param) return MW_ERR_UNSUPPORTED;
  net->apply_params = params;
  net->apply_lr = (float)lr;
  const mw_status r = mw_forward_sweep(net, params, x, g0, params_out, workspace, workspace_bytes, stream);
  net->apply_params = nullptr;
  return r;
}

extern "C" mw_status mw_backprop_reference(mw_net* net, const void* const* params, const void* x,
                                           const void* loss_target, void* const* dW_out,
                                           double* loss_out, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  if (!net || !params || !x || !loss_target || !dW_out) return MW_ERR_INVALID_ARG;
  for (int l = 0; l < net->L; ++l)
    if (!params[l]) return MW_ERR_INVALID_ARG;
  MW_TRY(check_ws(workspace, workspace_bytes, net->bpl.total));
  cudaStream_t s = (cudaStream_t)stream;
  if (net->ws_done == workspace) net->ws_done = nullptr;  // the stores are overwritten
  if (net->warm_ws == workspace) net->warm_ws = nullptr;
  if (net->backend == MW_BACKEND_TENSOR)
    return tensor_backprop(net, params, x, loss_target, dW_out, loss_out, workspace, s);
  if (net->opts.prec == MW_F64)
    return simt_backprop<double>(net, params, (const double*)x, loss_target, dW_out, loss_out,
                                 workspace, s);
  return simt_backprop<float>(net, params, (const float*)x, loss_target, dW_out, loss_out,
                              workspace, s);
}

extern "C" mw_status mw_export_masks(const mw_net* net, const void* workspace, int32_t layer,
                                     uint32_t* host_words, size_t host_words_capacity,
                                     int32_t* rows_out, int32_t* words_per_row_out, void* stream) {
  if (!net || !workspace || !host_words || layer < 0 || layer >= net->L) return MW_ERR_INVALID_ARG;
  const LayerInfo& li = net->info[layer];
  const size_t nw = (size_t)li.rows * li.wpr;
  if (host_words_capacity < nw) return MW_ERR_INVALID_ARG;
  if (rows_out) *rows_out = (int32_t)li.rows;
  if (words_per_row_out) *words_per_row_out = li.wpr;
  cudaStream_t s = (cudaStream_t)stream;
  // the mask regions sit at the same offsets in both layouts
  const char* src = static_cast<const char*>(workspace) + net->mwl.mask[layer].off;
  MW_CUDA_OK(cudaMemcpyAsync(host_words, src, nw * sizeof(uint32_t), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return MW_OK;
}

extern "C" mw_status mw_last_device_status(const mw_net* net, void* workspace, void* stream,
                                           uint32_t detail[4]) {
  if (!net || !workspace) return MW_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  DeviceStatus host;
  MW_CUDA_OK(cudaMemcpyAsync(&host, workspace, sizeof(host), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  if (detail) std::memcpy(detail, host.detail, sizeof(host.detail));
  if (host.code != 0) {
    // whatever failed, inverses kept in this workspace are no longer trusted
    if (net->warm_ws == workspace) const_cast<mw_net*>(net)->warm_ws = nullptr;
    MW_CUDA_OK(cudaMemsetAsync(workspace, 0, sizeof(DeviceStatus), s));
    MW_CUDA_OK(cudaStreamSynchronize(s));
  }
  return host.code <= MW_ERR_CUDA ? (mw_status)host.code : MW_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------
// stand-alone kernels
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_pack_sign_bits(const void* z, int32_t dtype, int64_t rows, int32_t cols,
                                       uint32_t* words, void* stream) {
  if (rows < 0 || cols < 0) return MW_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return MW_OK;
  if (!z || !words) return MW_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  switch (dtype) {
    case 0: return pack_sign_bits<double>((const double*)z, rows, cols, words, s);
    case 1: return pack_sign_bits<float>((const float*)z, rows, cols, words, s);
    case 2: return pack_sign_bits<__nv_bfloat16>((const __nv_bfloat16*)z, rows, cols, words, s);
  }
  return MW_ERR_INVALID_ARG;
}

extern "C" mw_status mw_relu_fragment_compact(const float* h, const uint32_t* words, int64_t rows,
                                              int32_t cols, uint32_t* cnt, uint32_t* off,
                                              float* vals, uint32_t* total_out, void* scratch,
                                              size_t scratch_bytes, void* stream) {
  if (rows < 0 || cols < 0) return MW_ERR_INVALID_ARG;
  if (rows == 0) return MW_OK;
  if (!h || !words || !cnt || !off || !vals) return MW_ERR_INVALID_ARG;
  if ((int64_t)rows * cols >= ((int64_t)1 << 32)) return MW_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  MW_TRY(fragment_offsets(words, rows, cols, cnt, off, total_out, scratch, scratch_bytes, s));
  return fragment_compact<float>(h, words, rows, cols, off, vals, s);
}

extern "C" mw_status mw_activation_vijp(const float* gz, const uint32_t* words, int64_t rows,
                                        int32_t cols, int32_t act, float slope, const uint32_t* off,
                                        const float* vals, float* h_out, float* gz_out,
                                        void* stream) {
  if (rows < 0 || cols < 0 || act < MW_ACT_NONE || act > MW_ACT_RELU) return MW_ERR_INVALID_ARG;
  if (rows == 0 || cols == 0) return MW_OK;
  if (!gz || !words || !h_out) return MW_ERR_INVALID_ARG;
  if (act == MW_ACT_LEAKY_RELU && !(slope != 0.f)) return MW_ERR_INVALID_ARG;
  return activation_vijp<float>(gz, words, rows, cols, act, (double)slope, off, vals, h_out, gz_out,
                                (cudaStream_t)stream);
}

// ---------------------------------------------------------------------------------------
// whole step from host buffers, and measurement hooks
// ---------------------------------------------------------------------------------------
extern "C" mw_status mw_gradient_step_host(mw_net* net, const void* const* params,
                                           const void* x_host, size_t x_bytes,
                                           const void* target_host, size_t target_bytes,
                                           void* x_dev, void* target_dev, void* g0_dev,
                                           void* const* dW_out, double* loss_dev,
                                           double* loss_host, void* workspace,
                                           size_t workspace_bytes, void* stream) {
  if (!net || !x_host || !target_host || !x_dev || !target_dev || !loss_dev || !loss_host)
    return MW_ERR_INVALID_ARG;   // g0_dev: as g0_out of mw_input_cotangent
  cudaStream_t s = (cudaStream_t)stream;
  MW_CUDA_OK(cudaMemcpyAsync(x_dev, x_host, x_bytes, cudaMemcpyHostToDevice, s));
  MW_CUDA_OK(cudaMemcpyAsync(target_dev, target_host, target_bytes, cudaMemcpyHostToDevice, s));
  MW_TRY(mw_input_cotangent(net, params, x_dev, target_dev, g0_dev, loss_dev, workspace,
                            workspace_bytes, stream));
  MW_TRY(mw_forward_sweep(net, params, x_dev, g0_dev, dW_out, workspace, workspace_bytes, stream));
  MW_CUDA_OK(cudaMemcpyAsync(loss_host, loss_dev, sizeof(double), cudaMemcpyDeviceToHost, s));
  MW_CUDA_OK(cudaStreamSynchronize(s));
  return MW_OK;
}

extern "C" int64_t mw_launch_count(void) { return (int64_t)g_launch_count; }

extern "C" int32_t mw_set_pair_mode(int32_t enable) { return tc_set_pair_mode(enable); }
extern "C" int32_t mw_set_merge_orders(int32_t enable) { return tc_set_merge_orders(enable); }
extern "C" int32_t mw_set_cooperative_launch(int32_t enable) { return tc_set_cooperative(enable); }
extern "C" int32_t mw_set_bulk_epilogue(int32_t enable) { return tc_set_bulk_epilogue(enable); }
namespace mw {
int g_sweep_chains = 1;
}
extern "C" int32_t mw_set_sweep_chains(int32_t enable) {
  const int32_t old = mw::g_sweep_chains;
  mw::g_sweep_chains = enable < 0 ? 0 : enable > 2 ? 2 : enable;
  return old;
}

extern "C" void mw_profile_begin(void) { tc_profile_begin(); }

extern "C" mw_status mw_profile_end(double* total_ms, int64_t* launches, double* flops,
                                    double* mma_flops) {
  long long n = 0;
  mw_status r = tc_profile_end(total_ms, &n, flops, mma_flops);
  if (launches) *launches = (int64_t)n;
  return r;
}
