// Host-side network description and workspace layout (internal).
#pragma once
#include <vector>

#include "mw_common.cuh"

namespace mw {

struct LayerInfo {
  int64_t rows;        // B (dense, head) or B*H*W (conv): rows of the [rows][cols] view of z
  int cols;            // n_out (dense, head) or C_out (conv)
  int wpr;             // mask words per row
  int64_t in_elems;    // elements of x_{l-1}
  int64_t out_elems;   // elements of x_l
  int64_t w_elems;     // elements of the weight
  int inv_n;           // size of the square block that is inverted (n, or C for conv), 0 for head
};

struct Region {
  size_t off = 0, bytes = 0;
};

struct Layout {
  size_t total = 0;
  size_t residual = 0;  // bytes that must survive between the phases
  Region status, partials;
  std::vector<Region> mask, frag_cnt, frag_off, frag_rank, frag_vals, reseed, stored_act;
  Region frag_total, h_last;
  Region act[2], cot[2], z, gz, aux0, aux1;  // aux: conv vijp iterate / h', wgrad partials
  std::vector<Region> inv;                   // per layer (resident) or all the same slot
  Region inv_scratch;
  // tensor-core backend operands (bf16 term planes)
  std::vector<Region> w_planes;              // split weights (MW_F32), per layer or one slot
  Region xp[5], hp[2], gzp[4], ns_r, ns_x, ns_w; // activation / cotangent / g_z planes (rings), NS scratch
  // convolution nets on the tensor cores
  std::vector<Region> cw, cwhat, cwinv;      // per layer: kernel, folded kernel, centre-tap inverse (term planes)
  std::vector<Region> cfrag;                 // per layer: fragmental checkpoints of a 1-D convolution
  Region cwinv_f32, cwhat_f32, cg[2], chpf, cxf, cpart, clogits, cseed;
  Region ns_sumsq, ns_scale;
  Region prog_table[3], prog_done[3];        // product tables and completion counters of program launches
  Region split[3];                           // K-split meeting places of concurrently running products
  // LU-parameterised dense nets: term planes of one layer's L, U, L^-1, U^-1, two block-substitution
  // temporaries, the planes of one gradient, two fp32 products of the gradient's chain rule, and
  // the inverted diagonal blocks of every layer (fp32)
  Region lu_l, lu_u, lu_t, lu_s, lu_y[2], lu_g, lu_a, lu_b, lu_diag;
  Region lu_table, lu_done;                  // product table and counters of the factor-preparation program
};

}  // namespace mw

struct mw_net {
  std::vector<mw_layer_desc> layers;
  std::vector<mw::LayerInfo> info;
  int L = 0, B = 0;
  mw_net_opts opts{};
  int backend = MW_BACKEND_SIMT;
  size_t es = 4;   // bytes of the working scalar (8 for MW_F64)
  mw::Layout mwl, bpl;
  // state
  const void* ws_done = nullptr;   // workspace that holds a finished Phase I+II
  const void* x_done = nullptr;
  void* tc = nullptr;              // tensor-core backend private state
  bool lean_seed = false;          // the net can keep the sweep's seed itself (g0 optional)
  // warm_inverse nets: the workspace whose kept inverses the next mw_input_cotangent may refresh
  // (nullptr: none, the next call computes them from scratch), and which of the two homes of the
  // Newton-Schulz iterate holds the current inverse
  const void* warm_ws = nullptr;
  int inv_side = 0;
  // mw_forward_sweep_apply in progress: the weight vjp's epilogue writes theta - apply_lr * g
  // (theta = apply_params[l]) instead of g
  const void* const* apply_params = nullptr;
  float apply_lr = 0.f;
  // mw_sweep_bucket_events: the forward sweep records bucket_events[b] on its stream once the
  // gradients of layers [b * bucket_layers, (b + 1) * bucket_layers) are enqueued
  std::vector<cudaEvent_t> bucket_events;
  int bucket_layers = 0;
  int buckets_recorded = 0;     // during a sweep: events already recorded
};

namespace mw {
// called by a sweep after the launch that completes the gradients of all layers < done_layers
inline void record_buckets(mw_net* n, int done_layers, cudaStream_t s) {
  if (n->bucket_layers <= 0) return;
  const int nb = (int)n->bucket_events.size();
  while (n->buckets_recorded < nb) {
    const int last = (n->buckets_recorded + 1) * n->bucket_layers;      // one past the bucket's last layer
    if ((last < n->L ? last : n->L) > done_layers) break;
    cudaEventRecord(n->bucket_events[(size_t)n->buckets_recorded], s);
    ++n->buckets_recorded;
  }
}
inline bool is_reseed(const mw_net* n, int l_out) {   // l_out = index of x_l / h_l, 1..L-1
  const int K = n->opts.reseed_every;
  return K > 0 && l_out > 0 && l_out < n->L && (l_out % K) == 0;
}
template <typename T>
inline T* at(void* ws, const Region& r) { return reinterpret_cast<T*>(static_cast<char*>(ws) + r.off); }
inline DeviceStatus* status_of(void* ws, const Layout& l) { return at<DeviceStatus>(ws, l.status); }
}  // namespace mw
