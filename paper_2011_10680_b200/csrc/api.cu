// C ABI of libhq.so: argument validation, dispatch to the kernels, and the table-driven network
// runner.  Host code only; every step of the inference path runs in the kernels of the other
// translation units.
#include <new>
#include <vector>

#include "hq_internal.cuh"

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline bool type_range_ok(int bits, int is_signed, int qmin, int qmax) {
  long long lo, hi;
  if (bits == 32) { lo = -(1LL << 31); hi = (1LL << 31) - 1; }
  else if (is_signed) { lo = -(1LL << (bits - 1)); hi = (1LL << (bits - 1)) - 1; }
  else { lo = 0; hi = (1LL << bits) - 1; }
  return qmin <= qmax && qmin >= lo && qmax <= hi;
}

inline hq_status check_tensor(const hq_tensor* t, bool allow4, bool allow8, bool allow32) {
  if (!t || !t->data) return HQ_ERR_INVALID_ARG;
  if (t->n < 0 || t->h < 1 || t->w < 1 || t->c < 1) return HQ_ERR_INVALID_ARG;
  if (!((t->bits == 4 && allow4) || (t->bits == 8 && allow8) || (t->bits == 32 && allow32))) return HQ_ERR_INVALID_ARG;
  if (t->bits == 4 && (t->c & 1)) return HQ_ERR_INVALID_ARG;
  if (!aligned16(t->data)) return HQ_ERR_ALIGNMENT;
  return HQ_OK;
}

inline long long tensor_bytes(int n, int h, int w, int c, int bits) {
  return (long long)n * h * w * c * bits / 8;
}

// `scratch` / `scratch_bytes`: buffer for the lowered first-layer path owned by the caller (a
// network); NULL means use (and if needed grow) the handle's own buffer.
hq_status conv_common(hq_handle* h, const hq_tensor* in, const hq_conv_desc* d, hq_tensor* out, void* stream,
                      void* scratch = nullptr, size_t scratch_bytes = 0, const void* res_narrow = nullptr,
                      const void* wgt_widened = nullptr) {
  if (!h || !d) return HQ_ERR_INVALID_ARG;
  hq_status st = check_tensor(in, true, true, false);
  if (st != HQ_OK) return st;
  st = check_tensor(out, true, true, true);
  if (st != HQ_OK) return st;
  if (d->kh < 1 || d->kw < 1 || d->stride < 1 || d->pad < 0 || d->cin < 1 || d->cout < 1) return HQ_ERR_INVALID_ARG;
  if (d->cin != in->c || d->w_bits != in->bits || !d->w) return HQ_ERR_INVALID_ARG;
  if (in->h + 2 * d->pad < d->kh || in->w + 2 * d->pad < d->kw) return HQ_ERR_INVALID_ARG;
  const int ho = (in->h + 2 * d->pad - d->kh) / d->stride + 1;
  const int wo = (in->w + 2 * d->pad - d->kw) / d->stride + 1;
  if (out->n != in->n || out->h != ho || out->w != wo || out->c != d->cout) return HQ_ERR_INVALID_ARG;
  if (!aligned16(d->w)) return HQ_ERR_ALIGNMENT;
  if (out->bits == 32) {
    if (d->residual) return HQ_ERR_INVALID_ARG;
  } else {
    if (!d->requant.b || !d->requant.c) return HQ_ERR_INVALID_ARG;
    if (!type_range_ok(out->bits, out->is_signed, d->qmin, d->qmax)) return HQ_ERR_INVALID_ARG;
    if (d->residual) {
      const hq_tensor* r = d->residual;
      st = check_tensor(r, false, true, true);
      if (st != HQ_OK) return st;
      if (r->n != out->n || r->h != out->h || r->w != out->w || r->c != out->c) return HQ_ERR_INVALID_ARG;
      if (!d->res_rescale.b || !d->res_rescale.c) return HQ_ERR_INVALID_ARG;
    }
  }
  ConvArgs a{};
  a.in = in->data; a.n = in->n; a.h = in->h; a.w = in->w; a.cin = in->c; a.in_bits = in->bits; a.in_signed = in->is_signed;
  a.wgt = d->w; a.wgt_widened = wgt_widened; a.cout = d->cout; a.kh = d->kh; a.kw = d->kw; a.stride = d->stride; a.pad = d->pad;
  a.bias = d->bias; a.b = d->requant.b; a.c = d->requant.c;
  if (d->residual && out->bits != 32) {
    a.res = d->residual->data; a.res_bits = d->residual->bits; a.res_signed = d->residual->is_signed;
    a.rb = d->res_rescale.b; a.rc = d->res_rescale.c;
    a.res_narrow = res_narrow;
  }
  a.relu = d->relu; a.qmin = d->qmin; a.qmax = d->qmax;
  a.out = out->data; a.ho = ho; a.wo = wo; a.out_bits = out->bits; a.out_signed = out->is_signed;
  cudaStream_t s = (cudaStream_t)stream;
  const bool tc_ok = hq_conv_tc_supported(a);
  const bool force_tc = h->conv_path >= 2;
  if (force_tc && !tc_ok && !hq_conv_widen4_applies(a)) return HQ_ERR_UNSUPPORTED;
  // Scratch for a lowered form: the caller's buffer (a network sized it when it was built), else the handle's own,
  // grown here.  A failure to grow it (e.g. inside a stream capture) is remembered and returned when tensor cores
  // were demanded; in automatic mode the CUDA-core kernel below takes the layer instead.
  hq_status scratch_err = HQ_OK;
  auto scratch_for = [&](size_t need) -> void* {
    if (scratch) return scratch_bytes >= need ? scratch : nullptr;
    const hq_status st = hq_reserve_workspace(h, need, s);
    if (st != HQ_OK) { scratch_err = st; return nullptr; }
    return h->workspace;
  };
  if (h->conv_path != 1 && tc_ok) {
    // A single large call with an 8-bit residual: its narrow residual pairs are worked out first, in the handle's
    // buffer (a network prepares them once when it is built); one small launch that the cheaper epilogue repays.
    if (a.res && a.res_bits == 8 && !a.res_narrow && a.cout <= kNarrowChannels &&
        (long long)a.n * ho * wo * a.cout >= (1ll << 25) &&
        hq_launch_residual_narrow(a.rb, a.rc, a.res_signed, a.cout, h->narrow_pairs, s) == cudaSuccess) {
      a.res_narrow = h->narrow_pairs;
      a.res_narrow_fresh = 1;
    }
    const hq_status st = hq_launch_conv_tc(h, a, s);
    if (st != HQ_ERR_UNSUPPORTED) return st;
    // declined before anything was launched (an im2col fetch from a tensor below 128 KiB, more channel tiles than
    // SMs): the patch-matrix form still runs the contraction on the tensor cores
    if (hq_conv_lowering_applies(a)) {
      if (void* buf = scratch_for(hq_conv_lowering_bytes(a))) { const hq_status st2 = hq_launch_conv_lowered(h, a, buf, s); if (st2 != HQ_ERR_UNSUPPORTED || force_tc) return st2; }
    }
    if (force_tc) return scratch_err != HQ_OK ? scratch_err : HQ_ERR_UNSUPPORTED;
  } else if (h->conv_path != 1) {
    if (hq_conv_widen4_applies(a)) {
      // packed 4-bit operands: widened copies in scratch, then the tensor-core kernel
      if (void* buf = scratch_for(hq_conv_widen4_bytes(a))) { const hq_status st2 = hq_launch_conv_widen4(h, a, buf, s); if (st2 != HQ_ERR_UNSUPPORTED || force_tc) return st2; }
      if (force_tc) return scratch_err != HQ_OK ? scratch_err : HQ_ERR_WORKSPACE;
    } else if (hq_conv_s2d_applies(a)) {
      // ImageNet-style first layer: space-to-depth copy of the image, then the tensor-core kernel
      if (void* buf = scratch_for(hq_conv_s2d_bytes(a))) { const hq_status st2 = hq_launch_conv_s2d(h, a, buf, s); if (st2 != HQ_ERR_UNSUPPORTED || force_tc) return st2; }
    } else if (hq_conv_lowering_applies(a)) {
      // thin first layers: patch matrix in scratch, then the tensor-core kernel
      if (void* buf = scratch_for(hq_conv_lowering_bytes(a))) { const hq_status st2 = hq_launch_conv_lowered(h, a, buf, s); if (st2 != HQ_ERR_UNSUPPORTED || force_tc) return st2; }
    }
  }
  return hq_launch_conv_cuda_core(a, s) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

}  // namespace

hq_status hq_reserve_workspace(hq_handle* h, size_t bytes, cudaStream_t s) {
  if (bytes <= h->workspace_bytes) return HQ_OK;
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess || cap != cudaStreamCaptureStatusNone) return HQ_ERR_WORKSPACE;
  // the old buffer may still be read by queued work
  if (cudaDeviceSynchronize() != cudaSuccess) return HQ_ERR_CUDA;
  if (h->workspace) { cudaFree(h->workspace); h->workspace = nullptr; h->workspace_bytes = 0; }
  if (cudaMalloc(&h->workspace, bytes) != cudaSuccess) { cudaGetLastError(); return HQ_ERR_WORKSPACE; }
  h->workspace_bytes = bytes;
  return HQ_OK;
}

// ------------------------------------------------------------------------------------------------
// Every buffer a network owns sits between two guard bands of kGuardBytes bytes filled with kGuardByte when the
// network is built.  No kernel may touch them: hq_network_check_guards reads them back, which is how the tests look
// for writes beyond a tensor (before its first or after its last byte) on the buffers the caller never sees.
constexpr size_t kGuardBytes = 256;
constexpr int kGuardByte = 0xA5;
struct GuardedBuffer { void* base; void* data; size_t bytes; int32_t layer; };

struct hq_network {
  hq_handle* h;
  std::vector<GuardedBuffer> buffers; // every device allocation of the network, with its guard bands
  std::vector<hq_layer> layers;
  std::vector<hq_tensor> outs;       // planned output tensor of every layer (data owned by the network)
  std::vector<long long> bytes;
  int32_t batch, image_h, image_w, image_c, image_signed;
  int32_t launches;
  std::vector<void*> res_narrow;     // per conv layer with a fused 8-bit residual: its narrow residual pairs (owned)
  std::vector<void*> narrow0, narrow1; // per ADD / REQUANT layer with 8-bit operands: narrow pairs of the two branches (owned)
  std::vector<void*> wgt_widened;    // per 4-bit conv layer on the tensor-core path: its weights, one byte per value (owned)
  std::vector<char> stored_wide;     // per layer: its 4-bit output is kept one value per byte (all consumers are such convs)
  std::vector<char> tile_order;      // per conv / linear / concat layer: tensors walked from the last pixel to the first (see plan_tile_orders)
  void* scratch;                     // patch matrix of the lowered first layer (owned)
  size_t scratch_bytes;
  // graph cache: one instantiated graph per (images, logits) pointer pair, a few pairs kept so
  // that double-buffered callers do not re-capture every step
  struct CachedGraph { cudaGraphExec_t exec; const void* images; void* logits; };
  std::vector<CachedGraph> graphs;
};

// Order in which every convolution (and concatenation) walks its tensors.  At large batch a layer's tensors exceed the
// L2, which still holds what the launch before wrote LAST; a consumer that starts at the same end reads that part
// without going to HBM.  So a convolution runs opposite to the layer that produced its main input, except when the
// layer right after it is an element-wise or pooling kernel reading its output (those always run first to last): then
// it runs last to first for that kernel's sake.  A concatenation runs opposite to the launch right before it (the
// pooling branch's window sums in an Inception module).  The arithmetic does not depend on the order.
static void plan_tile_orders(hq_network* net) {
  const int n = (int)net->layers.size();
  net->tile_order.assign(n, 0);
  auto is_conv = [&](int i) { return net->layers[i].op == HQ_OP_CONV || net->layers[i].op == HQ_OP_LINEAR; };
  auto either_way = [&](int i) { return is_conv(i) || net->layers[i].op == HQ_OP_CONCAT; };
  for (int i = 0; i < n; ++i) {
    if (!either_way(i)) continue;
    char order;
    if (!is_conv(i)) {
      order = i > 0 ? !net->tile_order[i - 1] : 0;
    } else {
      const int src = net->layers[i].in0;
      order = src < 0 ? 0 : !net->tile_order[src];
    }
    if (i + 1 < n && !either_way(i + 1) && net->layers[i + 1].in0 == i) order = 1;
    net->tile_order[i] = order;
  }
}

// Allocate `bytes` for layer `layer` of `net` between two guard bands; NULL when the device is out of memory.
static void* net_alloc(hq_network* net, size_t bytes, int32_t layer) {
  unsigned char* base = nullptr;
  if (cudaMalloc(&base, bytes + 2 * kGuardBytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (cudaMemset(base, kGuardByte, kGuardBytes) != cudaSuccess ||
      cudaMemset(base + kGuardBytes + bytes, kGuardByte, kGuardBytes) != cudaSuccess) { cudaFree(base); return nullptr; }
  net->buffers.push_back({base, base + kGuardBytes, bytes, layer});
  return base + kGuardBytes;
}

static void net_free(hq_network* net, void* data) {
  for (auto it = net->buffers.begin(); it != net->buffers.end(); ++it)
    if (it->data == data) { cudaFree(it->base); net->buffers.erase(it); return; }
}

extern "C" {

const char* hq_status_string(hq_status s) {
  switch (s) {
    case HQ_OK: return "HQ_OK";
    case HQ_ERR_INVALID_ARG: return "HQ_ERR_INVALID_ARG";
    case HQ_ERR_UNSUPPORTED: return "HQ_ERR_UNSUPPORTED";
    case HQ_ERR_ALIGNMENT: return "HQ_ERR_ALIGNMENT";
    case HQ_ERR_RANGE: return "HQ_ERR_RANGE";
    case HQ_ERR_WORKSPACE: return "HQ_ERR_WORKSPACE";
    case HQ_ERR_CUDA: return "HQ_ERR_CUDA";
    case HQ_ERR_TIMEOUT: return "HQ_ERR_TIMEOUT";
    case HQ_ERR_INFEASIBLE: return "HQ_ERR_INFEASIBLE";
  }
  return "HQ_ERR_UNKNOWN";
}

hq_status hq_create(int32_t device, hq_handle** out) {
  if (!out) return HQ_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess) return HQ_ERR_CUDA;
  if (device < 0 || device >= count) return HQ_ERR_INVALID_ARG;
  if (cudaSetDevice(device) != cudaSuccess) return HQ_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return HQ_ERR_CUDA;
  if (prop.major != 10) return HQ_ERR_UNSUPPORTED;       // kernels are built for sm_100a only
  hq_handle* h = new (std::nothrow) hq_handle();
  if (!h) return HQ_ERR_WORKSPACE;
  h->device = device;
  h->conv_path = 0;
  h->tile_order = 0;
  h->sm_count = prop.multiProcessorCount;
  h->workspace = nullptr;
  h->workspace_bytes = 0;
  if (!hq_conv_tc_init()) { delete h; return HQ_ERR_CUDA; }
  if (cudaMalloc(&h->dev_status, sizeof(uint32_t)) != cudaSuccess) { delete h; return HQ_ERR_WORKSPACE; }
  if (cudaMemset(h->dev_status, 0, sizeof(uint32_t)) != cudaSuccess) { cudaFree(h->dev_status); delete h; return HQ_ERR_CUDA; }
  if (cudaMalloc(&h->narrow_pairs, (size_t)2 * kNarrowChannels * 16) != cudaSuccess) {
    cudaFree(h->dev_status); delete h; return HQ_ERR_WORKSPACE;
  }
  *out = h;
  return HQ_OK;
}

hq_status hq_destroy(hq_handle* h) {
  if (!h) return HQ_ERR_INVALID_ARG;
  cudaFree(h->dev_status);
  cudaFree(h->narrow_pairs);
  if (h->workspace) cudaFree(h->workspace);
  delete h;
  return HQ_OK;
}

hq_status hq_set_conv_path(hq_handle* h, int32_t path) {
  if (!h || path < 0 || path > 3) return HQ_ERR_INVALID_ARG;
  h->conv_path = path;
  return HQ_OK;
}

hq_status hq_set_tile_order(hq_handle* h, int32_t order) {
  if (!h || order < 0 || order > 1) return HQ_ERR_INVALID_ARG;
  h->tile_order = order;
  return HQ_OK;
}

hq_status hq_expire_wait_selftest(hq_handle* h, int32_t budget_ms, void* stream) {
  if (!h || budget_ms < 1 || budget_ms > 2000) return HQ_ERR_INVALID_ARG;
  return hq_launch_expire_wait(h->dev_status, budget_ms, (cudaStream_t)stream) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

hq_status hq_sync(hq_handle* h, void* stream) {
  if (!h) return HQ_ERR_INVALID_ARG;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HQ_ERR_CUDA;
  uint32_t word = 0;
  if (cudaMemcpy(&word, h->dev_status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return HQ_ERR_CUDA;
  if (word != 0) {
    cudaMemset(h->dev_status, 0, sizeof(uint32_t));
    return HQ_ERR_TIMEOUT;
  }
  return HQ_OK;
}

hq_status hq_conv2d(hq_handle* h, const hq_tensor* in, const hq_conv_desc* desc, hq_tensor* out, void* stream) {
  return conv_common(h, in, desc, out, stream);
}

hq_status hq_linear(hq_handle* h, const hq_tensor* in, const hq_conv_desc* d, hq_tensor* out, void* stream) {
  if (!in || !d || !out) return HQ_ERR_INVALID_ARG;
  if (d->kh != 1 || d->kw != 1 || d->stride != 1 || d->pad != 0 || d->residual) return HQ_ERR_INVALID_ARG;
  if (in->h != 1 || in->w != 1) return HQ_ERR_INVALID_ARG;
  return conv_common(h, in, d, out, stream);
}

static hq_status residual_add_impl(hq_handle* h, const hq_tensor* main_t, hq_dyadic mr, const hq_tensor* res, hq_dyadic rr,
                                   int32_t relu, int32_t qmin, int32_t qmax, hq_tensor* out, void* stream,
                                   const void* m_narrow, const void* r_narrow) {
  if (!h) return HQ_ERR_INVALID_ARG;
  hq_status st = check_tensor(main_t, true, true, true);
  if (st != HQ_OK) return st;
  st = check_tensor(out, true, true, true);
  if (st != HQ_OK) return st;
  if (out->n != main_t->n || out->h != main_t->h || out->w != main_t->w || out->c != main_t->c) return HQ_ERR_INVALID_ARG;
  if (!mr.b || !mr.c) return HQ_ERR_INVALID_ARG;
  if (!type_range_ok(out->bits, out->is_signed, qmin, qmax)) return HQ_ERR_INVALID_ARG;
  EltArgs a{};
  if (res) {
    st = check_tensor(res, true, true, true);
    if (st != HQ_OK) return st;
    if (res->n != out->n || res->h != out->h || res->w != out->w || res->c != out->c) return HQ_ERR_INVALID_ARG;
    if (!rr.b || !rr.c) return HQ_ERR_INVALID_ARG;
    a.res = res->data; a.res_bits = res->bits; a.res_signed = res->is_signed; a.rb = rr.b; a.rc = rr.c;
  }
  a.main_t = main_t->data; a.main_bits = main_t->bits; a.main_signed = main_t->is_signed; a.mb = mr.b; a.mc = mr.c;
  a.pixels = (long long)out->n * out->h * out->w; a.ch = out->c;
  a.relu = relu; a.qmin = qmin; a.qmax = qmax; a.out = out->data; a.out_bits = out->bits;
  a.m_narrow = m_narrow; a.r_narrow = r_narrow;
  a.status = h->dev_status;
  // A single large call on 8-bit operands: the narrow pairs of both branches are worked out first, in the handle's
  // buffer (a network prepares them once when it is built).  One small launch that the cheaper arithmetic repays.
  cudaStream_t s = (cudaStream_t)stream;
  if (!m_narrow && main_t->bits == 8 && (!res || res->bits == 8) && out->c <= kNarrowChannels &&
      a.pixels * a.ch >= (1ll << 25)) {
    char* base = (char*)h->narrow_pairs;
    char* base1 = res ? base + (size_t)kNarrowChannels * 16 : nullptr;
    if (hq_launch_residual_narrow2(a.mb, a.mc, a.main_signed, base, a.rb, a.rc, a.res_signed, base1, a.ch, s) != cudaSuccess)
      return HQ_ERR_CUDA;
    a.m_narrow = base;
    a.r_narrow = base1;
  }
  return hq_launch_residual_add(a, h->sm_count, s) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

hq_status hq_residual_add(hq_handle* h, const hq_tensor* main_t, hq_dyadic mr, const hq_tensor* res, hq_dyadic rr,
                          int32_t relu, int32_t qmin, int32_t qmax, hq_tensor* out, void* stream) {
  return residual_add_impl(h, main_t, mr, res, rr, relu, qmin, qmax, out, stream, nullptr, nullptr);
}

hq_status hq_avgpool_requant(hq_handle* h, const hq_tensor* in, hq_dyadic r, int32_t qmin, int32_t qmax,
                             hq_tensor* out, void* stream) {
  if (!h) return HQ_ERR_INVALID_ARG;
  hq_status st = check_tensor(in, true, true, true);
  if (st != HQ_OK) return st;
  st = check_tensor(out, true, true, false);
  if (st != HQ_OK) return st;
  if (out->n != in->n || out->h != 1 || out->w != 1 || out->c != in->c) return HQ_ERR_INVALID_ARG;
  if (!r.b || !r.c) return HQ_ERR_INVALID_ARG;
  if (!type_range_ok(out->bits, out->is_signed, qmin, qmax)) return HQ_ERR_INVALID_ARG;
  if ((long long)in->h * in->w > (1LL << 23)) return HQ_ERR_UNSUPPORTED;   // INT32 sum of 8-bit values
  return hq_launch_avgpool(in->data, in->n, in->h, in->w, in->c, in->bits, in->is_signed, r.b, r.c, qmin, qmax,
                           out->data, out->bits, (cudaStream_t)stream) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

hq_status hq_maxpool(hq_handle* h, const hq_tensor* in, int32_t k, int32_t stride, int32_t pad, hq_tensor* out,
                     void* stream) {
  if (!h) return HQ_ERR_INVALID_ARG;
  hq_status st = check_tensor(in, false, true, true);
  if (st != HQ_OK) return st;
  st = check_tensor(out, false, true, true);
  if (st != HQ_OK) return st;
  if (in->bits != out->bits) return HQ_ERR_INVALID_ARG;
  if (k < 1 || stride < 1 || pad < 0 || pad >= k) return HQ_ERR_INVALID_ARG;
  if (in->h + 2 * pad < k || in->w + 2 * pad < k) return HQ_ERR_INVALID_ARG;
  const int ho = (in->h + 2 * pad - k) / stride + 1, wo = (in->w + 2 * pad - k) / stride + 1;
  if (out->n != in->n || out->h != ho || out->w != wo || out->c != in->c || out->is_signed != in->is_signed)
    return HQ_ERR_INVALID_ARG;
  return hq_launch_maxpool(in->data, in->n, in->h, in->w, in->c, in->bits == 32 ? 32 : 8, in->is_signed, k, stride, pad,
                           out->data, ho, wo, (cudaStream_t)stream) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

// ------------------------------------------------------------------------------------------------
hq_status hq_network_create(hq_handle* h, const hq_layer* table, int32_t n_layers, int32_t batch,
                            int32_t image_h, int32_t image_w, int32_t image_c, int32_t image_signed,
                            hq_network** out) {
  if (!h || !table || !out || n_layers < 1 || batch < 1 || image_h < 1 || image_w < 1 || image_c < 1)
    return HQ_ERR_INVALID_ARG;
  *out = nullptr;
  hq_network* net = new (std::nothrow) hq_network();
  if (!net) return HQ_ERR_WORKSPACE;
  net->h = h; net->batch = batch;
  net->image_h = image_h; net->image_w = image_w; net->image_c = image_c; net->image_signed = image_signed;
  net->scratch = nullptr; net->scratch_bytes = 0;
  net->layers.assign(table, table + n_layers);
  net->outs.resize(n_layers);
  net->bytes.resize(n_layers);
  net->res_narrow.assign(n_layers, nullptr);
  net->wgt_widened.assign(n_layers, nullptr);
  net->stored_wide.assign(n_layers, 0);
  net->narrow0.assign(n_layers, nullptr);
  net->narrow1.assign(n_layers, nullptr);
  net->launches = n_layers;
  hq_status st = HQ_OK;
  auto shape_of = [&](int id, hq_tensor* t) -> bool {
    if (id == -1) { *t = hq_tensor{nullptr, batch, image_h, image_w, image_c, 8, image_signed}; return true; }
    if (id < 0) return false;
    *t = net->outs[id];
    return true;
  };
  for (int i = 0; i < n_layers && st == HQ_OK; ++i) {
    const hq_layer& l = net->layers[i];
    hq_tensor in{}, o{};
    if (l.in0 >= i || l.in1 >= i || !shape_of(l.in0, &in)) { st = HQ_ERR_INVALID_ARG; break; }
    o.n = batch; o.bits = l.out_bits; o.is_signed = l.out_signed;
    switch (l.op) {
      case HQ_OP_CONV: {
        const hq_conv_desc& d = l.conv;
        if (d.kh < 1 || d.kw < 1 || d.stride < 1 || d.pad < 0 || in.h + 2 * d.pad < d.kh || in.w + 2 * d.pad < d.kw) {
          st = HQ_ERR_INVALID_ARG; break;
        }
        o.h = (in.h + 2 * d.pad - d.kh) / d.stride + 1; o.w = (in.w + 2 * d.pad - d.kw) / d.stride + 1; o.c = d.cout;
        {
          ConvArgs a{};
          a.n = batch; a.h = in.h; a.w = in.w; a.cin = in.c; a.in_bits = in.bits; a.cout = d.cout; a.kh = d.kh; a.kw = d.kw;
          a.stride = d.stride; a.pad = d.pad; a.ho = o.h; a.wo = o.w; a.out_bits = o.bits;
          if (hq_conv_widen4_applies(a)) {
            const size_t need = hq_conv_widen4_bytes(a);
            if (need > net->scratch_bytes) net->scratch_bytes = need;
            net->launches += 1;                 // the activation-widening kernel (the weights are widened once, below)
            const long long wvals = (long long)d.cout * d.kh * d.kw * in.c;
            void* wbuf = net_alloc(net, (size_t)wvals, i);
            if (!wbuf) { st = HQ_ERR_WORKSPACE; break; }
            net->wgt_widened[i] = wbuf;
            if (hq_launch_widen_weights(d.w, wvals, wbuf, h->sm_count, nullptr) != cudaSuccess) { st = HQ_ERR_CUDA; break; }
          } else if (hq_conv_s2d_applies(a)) {
            const size_t need = hq_conv_s2d_bytes(a);
            if (need > net->scratch_bytes) net->scratch_bytes = need;
            net->launches += 1;                 // the space-to-depth kernel (the weights are re-laid out once, here)
            a.wgt = d.w; a.bias = d.bias; a.b = d.requant.b; a.c = d.requant.c;
            void* wbuf = net_alloc(net, hq_conv_s2d_prepared_bytes(a), i);
            if (!wbuf) { st = HQ_ERR_WORKSPACE; break; }
            net->wgt_widened[i] = wbuf;
            if (hq_prepare_conv_s2d(a, wbuf, nullptr) != cudaSuccess) { st = HQ_ERR_CUDA; break; }
          } else if ((!hq_conv_tc_supported(a) || hq_conv_tc_small_im2col(a)) && hq_conv_lowering_applies(a)) {
            const size_t need = hq_conv_lowering_bytes(a);
            if (need > net->scratch_bytes) net->scratch_bytes = need;
            net->launches += 2;                 // weight padding + patch matrix kernels
          }
        }
        break;
      }
      case HQ_OP_LINEAR:
        if (l.conv.cin != in.h * in.w * in.c) { st = HQ_ERR_INVALID_ARG; break; }
        o.h = 1; o.w = 1; o.c = l.conv.cout;
        break;
      case HQ_OP_MAXPOOL:
        if (l.pool_k < 1 || l.pool_stride < 1 || l.pool_pad < 0 || in.h + 2 * l.pool_pad < l.pool_k ||
            in.w + 2 * l.pool_pad < l.pool_k) { st = HQ_ERR_INVALID_ARG; break; }
        o.h = (in.h + 2 * l.pool_pad - l.pool_k) / l.pool_stride + 1;
        o.w = (in.w + 2 * l.pool_pad - l.pool_k) / l.pool_stride + 1; o.c = in.c;
        break;
      case HQ_OP_AVGPOOL: o.h = 1; o.w = 1; o.c = in.c; break;
      case HQ_OP_ADD: case HQ_OP_REQUANT: o.h = in.h; o.w = in.w; o.c = in.c; break;
      case HQ_OP_SUMPOOL:
        if (l.pool_k < 1 || l.pool_stride < 1 || l.pool_pad < 0 || l.pool_pad >= l.pool_k || in.h + 2 * l.pool_pad < l.pool_k ||
            in.w + 2 * l.pool_pad < l.pool_k || l.out_bits != 32) { st = HQ_ERR_INVALID_ARG; break; }
        o.h = (in.h + 2 * l.pool_pad - l.pool_k) / l.pool_stride + 1;
        o.w = (in.w + 2 * l.pool_pad - l.pool_k) / l.pool_stride + 1; o.c = in.c;
        break;
      case HQ_OP_CONCAT: {
        if (l.n_in < 1 || l.n_in > HQ_CONCAT_MAX_BRANCHES || l.in0 != l.ins[0]) { st = HQ_ERR_INVALID_ARG; break; }
        o.h = in.h; o.w = in.w; o.c = 0;
        for (int k = 0; k < l.n_in; ++k) {
          const int id = l.ins[k];
          if (id < 0 || id >= i || net->outs[id].h != in.h || net->outs[id].w != in.w) { st = HQ_ERR_INVALID_ARG; break; }
          o.c += net->outs[id].c;
        }
        break;
      }
      default: st = HQ_ERR_INVALID_ARG; break;
    }
    if (st != HQ_OK) break;
    if (!(o.bits == 4 || o.bits == 8 || o.bits == 32) || o.c < 1 || (o.bits == 4 && (o.c & 1))) { st = HQ_ERR_INVALID_ARG; break; }
    net->bytes[i] = tensor_bytes(o.n, o.h, o.w, o.c, o.bits);
    void* buf = net_alloc(net, (size_t)net->bytes[i], i);
    if (!buf) { st = HQ_ERR_WORKSPACE; break; }
    o.data = buf;
    net->outs[i] = o;
  }
  // A 4-bit tensor whose only readers are tensor-core convolutions (as their main input) is kept one value per
  // byte: its producer writes bytes clamped to the 4-bit range, the readers are plain 8-bit convolutions over
  // their widened weights, and no widening pass runs between them.  What leaves the network (layer taps, the
  // last layer) is packed.
  for (int i = 0; st == HQ_OK && i + 1 < n_layers; ++i) {
    const hq_layer& l = net->layers[i];
    if (net->outs[i].bits != 4) continue;
    if (l.op != HQ_OP_CONV && l.op != HQ_OP_REQUANT && l.op != HQ_OP_ADD) continue;
    if (((long long)net->outs[i].n * net->outs[i].h * net->outs[i].w * net->outs[i].c) % 8 != 0) continue;
    bool ok = false;
    for (int j = i + 1; j < n_layers; ++j) {
      const hq_layer& c = net->layers[j];
      if (c.in1 == i) { ok = false; break; }
      if (c.op == HQ_OP_CONCAT) {
        bool used = false;
        for (int k = 0; k < c.n_in; ++k) used = used || c.ins[k] == i;
        if (used) { ok = false; break; }
        continue;
      }
      if (c.in0 != i) continue;
      if (c.op != HQ_OP_CONV || !net->wgt_widened[j]) { ok = false; break; }
      ok = true;
    }
    if (!ok) continue;
    net->stored_wide[i] = 1;
    net_free(net, net->outs[i].data);
    const size_t wide = (size_t)net->outs[i].n * net->outs[i].h * net->outs[i].w * net->outs[i].c;
    void* buf = net_alloc(net, wide, i);
    net->outs[i].data = buf;
    if (!buf) { st = HQ_ERR_WORKSPACE; break; }
    for (int j = i + 1; j < n_layers; ++j)
      if (net->layers[j].in0 == i) net->launches -= 1;        // no activation-widening kernel ahead of this conv
  }
  if (st == HQ_OK && net->scratch_bytes) {
    const size_t want = net->scratch_bytes;
    net->scratch_bytes = 0;
    net->scratch = net_alloc(net, want, -1);
    if (!net->scratch) st = HQ_ERR_WORKSPACE;
    else net->scratch_bytes = want;
  }
  // narrow residual pairs of every conv with a fused 8-bit residual (a one-off search per channel)
  for (int i = 0; st == HQ_OK && i < n_layers; ++i) {
    const hq_layer& l = net->layers[i];
    if (l.op != HQ_OP_CONV || l.in1 < 0 || net->outs[l.in1].bits != 8 || net->outs[i].bits == 32) continue;
    if (!l.conv.res_rescale.b || !l.conv.res_rescale.c) continue;
    void* buf = net_alloc(net, (size_t)l.conv.cout * 16, i);
    if (!buf) { st = HQ_ERR_WORKSPACE; break; }
    net->res_narrow[i] = buf;
    if (hq_launch_residual_narrow(l.conv.res_rescale.b, l.conv.res_rescale.c, net->outs[l.in1].is_signed, l.conv.cout,
                                  buf, nullptr) != cudaSuccess) st = HQ_ERR_CUDA;
  }
  // ... and of the 8-bit branches of ADD / REQUANT layers
  for (int i = 0; st == HQ_OK && i < n_layers; ++i) {
    const hq_layer& l = net->layers[i];
    if (l.op != HQ_OP_ADD && l.op != HQ_OP_REQUANT) continue;
    const hq_tensor& t0 = (l.in0 >= 0) ? net->outs[l.in0] : net->outs[i];
    const int bits0 = l.in0 >= 0 ? t0.bits : 8, sgn0 = l.in0 >= 0 ? t0.is_signed : image_signed;
    const int ch = net->outs[i].c;
    if (bits0 != 8 || !l.rescale0.b || !l.rescale0.c) continue;
    if (l.op == HQ_OP_ADD && (l.in1 < 0 || net->outs[l.in1].bits != 8 || !l.rescale1.b || !l.rescale1.c)) continue;
    void* buf = net_alloc(net, (size_t)ch * 16, i);
    if (!buf) { st = HQ_ERR_WORKSPACE; break; }
    net->narrow0[i] = buf;
    if (hq_launch_residual_narrow(l.rescale0.b, l.rescale0.c, sgn0, ch, buf, nullptr) != cudaSuccess) { st = HQ_ERR_CUDA; break; }
    if (l.op == HQ_OP_ADD) {
      void* buf1 = net_alloc(net, (size_t)ch * 16, i);
      if (!buf1) { st = HQ_ERR_WORKSPACE; break; }
      net->narrow1[i] = buf1;
      if (hq_launch_residual_narrow(l.rescale1.b, l.rescale1.c, net->outs[l.in1].is_signed, ch, buf1, nullptr) != cudaSuccess) { st = HQ_ERR_CUDA; break; }
    }
  }
  if (st == HQ_OK) plan_tile_orders(net);
  if (st == HQ_OK && cudaDeviceSynchronize() != cudaSuccess) st = HQ_ERR_CUDA;
  if (st != HQ_OK) { hq_network_destroy(net); return st; }
  *out = net;
  return HQ_OK;
}

static hq_status run_layers(hq_network* net, const hq_tensor* images, hq_tensor* logits, void* const* taps,
                            cudaStream_t s, cudaEvent_t* marks = nullptr) {
  hq_handle* h = net->h;
  const int n_layers = (int)net->layers.size();
  for (int i = 0; i < n_layers; ++i) {
    if (marks && cudaEventRecord(marks[i], s) != cudaSuccess) return HQ_ERR_CUDA;
    const hq_layer& l = net->layers[i];
    hq_tensor in = (l.in0 == -1) ? *images : net->outs[l.in0];
    hq_tensor o = net->outs[i];
    if (i == n_layers - 1) o.data = logits->data;
    const bool in_wide = l.in0 >= 0 && net->stored_wide[l.in0];
    if (in_wide) in.bits = 8;                  // one value per byte
    if (net->stored_wide[i]) o.bits = 8;       // written as bytes clamped to the 4-bit range
    hq_status st = HQ_OK;
    switch (l.op) {
      case HQ_OP_CONV: case HQ_OP_LINEAR: {
        hq_conv_desc d = l.conv;
        hq_tensor res{};
        d.residual = nullptr;
        if (l.op == HQ_OP_CONV && l.in1 >= 0) { res = net->outs[l.in1]; d.residual = &res; }
        if (in_wide) { d.w_bits = 8; d.w = net->wgt_widened[i]; }
        const int32_t callers_order = h->tile_order;
        h->tile_order = net->tile_order[i];
        if (l.op == HQ_OP_LINEAR) { in.c = in.h * in.w * in.c; in.h = 1; in.w = 1; st = hq_linear(h, &in, &d, &o, s); }
        else st = conv_common(h, &in, &d, &o, s, net->scratch, net->scratch_bytes, net->res_narrow[i], in_wide ? nullptr : net->wgt_widened[i]);
        h->tile_order = callers_order;
        break;
      }
      case HQ_OP_MAXPOOL: st = hq_maxpool(h, &in, l.pool_k, l.pool_stride, l.pool_pad, &o, s); break;
      case HQ_OP_AVGPOOL: st = hq_avgpool_requant(h, &in, l.rescale0, l.qmin, l.qmax, &o, s); break;
      case HQ_OP_ADD: {
        if (l.in1 < 0) return HQ_ERR_INVALID_ARG;
        hq_tensor res = net->outs[l.in1];
        st = residual_add_impl(h, &in, l.rescale0, &res, l.rescale1, l.relu, l.qmin, l.qmax, &o, s, net->narrow0[i], net->narrow1[i]);
        break;
      }
      case HQ_OP_REQUANT: {
        hq_dyadic none{nullptr, nullptr};
        st = residual_add_impl(h, &in, l.rescale0, nullptr, none, l.relu, l.qmin, l.qmax, &o, s, net->narrow0[i], nullptr);
        break;
      }
      case HQ_OP_SUMPOOL: st = hq_sumpool(h, &in, l.pool_k, l.pool_stride, l.pool_pad, &o, s); break;
      case HQ_OP_CONCAT: {
        hq_tensor br[HQ_CONCAT_MAX_BRANCHES];
        for (int k = 0; k < l.n_in; ++k) br[k] = net->outs[l.ins[k]];
        const int32_t callers_order = h->tile_order;
        h->tile_order = net->tile_order[i];
        st = hq_concat_requant(h, l.n_in, br, l.rescales, l.relu, l.qmin, l.qmax, &o, s);
        h->tile_order = callers_order;
        break;
      }
      default: return HQ_ERR_INVALID_ARG;
    }
    if (st != HQ_OK) return st;
    if (taps && taps[i]) {
      if (net->stored_wide[i]) {
        if (hq_launch_pack4(o.data, (long long)o.n * o.h * o.w * o.c, taps[i], h->sm_count, s) != cudaSuccess) return HQ_ERR_CUDA;
      } else if (cudaMemcpyAsync(taps[i], o.data, (size_t)net->bytes[i], cudaMemcpyDeviceToDevice, s) != cudaSuccess) {
        return HQ_ERR_CUDA;
      }
    }
  }
  if (marks && cudaEventRecord(marks[n_layers], s) != cudaSuccess) return HQ_ERR_CUDA;
  return HQ_OK;
}

hq_status hq_network_time_layers(hq_network* net, const hq_tensor* images, hq_tensor* logits, int64_t* ns,
                                 void* stream) {
  if (!net || !images || !logits || !ns || !images->data || !logits->data) return HQ_ERR_INVALID_ARG;
  const int n_layers = (int)net->layers.size();
  std::vector<cudaEvent_t> marks(n_layers + 1, nullptr);
  hq_status st = HQ_OK;
  for (auto& e : marks) if (cudaEventCreate(&e) != cudaSuccess) st = HQ_ERR_CUDA;
  cudaStream_t s = (cudaStream_t)stream;
  if (st == HQ_OK) st = run_layers(net, images, logits, nullptr, s, marks.data());
  if (st == HQ_OK && cudaStreamSynchronize(s) != cudaSuccess) st = HQ_ERR_CUDA;
  for (int i = 0; i < n_layers && st == HQ_OK; ++i) {
    float ms = 0;   // timing only: not part of the integer pipeline
    if (cudaEventElapsedTime(&ms, marks[i], marks[i + 1]) != cudaSuccess) st = HQ_ERR_CUDA;
    ns[i] = (int64_t)(ms * 1.0e6f);
  }
  for (auto& e : marks) if (e) cudaEventDestroy(e);
  return st;
}

hq_status hq_run_network(hq_network* net, const hq_tensor* images, hq_tensor* logits, void* const* layer_taps,
                         void* stream) {
  if (!net || !images || !logits || !images->data || !logits->data) return HQ_ERR_INVALID_ARG;
  if (images->n != net->batch || images->h != net->image_h || images->w != net->image_w ||
      images->c != net->image_c || images->bits != 8 || images->is_signed != net->image_signed)
    return HQ_ERR_INVALID_ARG;
  const hq_tensor& last = net->outs.back();
  if (logits->n != last.n || logits->h != last.h || logits->w != last.w || logits->c != last.c ||
      logits->bits != last.bits) return HQ_ERR_INVALID_ARG;
  if (!aligned16(images->data) || !aligned16(logits->data)) return HQ_ERR_ALIGNMENT;
  cudaStream_t s = (cudaStream_t)stream;

  // Inside a caller's capture, or when taps are requested: plain launches.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(s, &cap) != cudaSuccess) return HQ_ERR_CUDA;
  if (cap != cudaStreamCaptureStatusNone || layer_taps || s == nullptr) return run_layers(net, images, logits, layer_taps, s);

  // Otherwise replay a CUDA graph of the whole table (captured once per (images, logits) pair).
  for (const auto& g : net->graphs)
    if (g.images == images->data && g.logits == logits->data)
      return cudaGraphLaunch(g.exec, s) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
  if (net->graphs.size() >= 4) {
    cudaGraphExecDestroy(net->graphs.front().exec);
    net->graphs.erase(net->graphs.begin());
  }
  if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return HQ_ERR_CUDA;
  const hq_status st = run_layers(net, images, logits, nullptr, s);
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(s, &graph);
  if (st != HQ_OK) { if (graph) cudaGraphDestroy(graph); return st; }
  if (e != cudaSuccess || !graph) return HQ_ERR_CUDA;
  cudaGraphExec_t exec = nullptr;
  const cudaError_t e2 = cudaGraphInstantiate(&exec, graph, 0);
  cudaGraphDestroy(graph);
  if (e2 != cudaSuccess || !exec) return HQ_ERR_CUDA;
  net->graphs.push_back({exec, images->data, logits->data});
  return cudaGraphLaunch(exec, s) == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}

hq_status hq_network_layer_bytes(const hq_network* net, int32_t layer, int64_t* bytes) {
  if (!net || !bytes || layer < 0 || layer >= (int)net->layers.size()) return HQ_ERR_INVALID_ARG;
  *bytes = net->bytes[layer];
  return HQ_OK;
}

hq_status hq_network_launch_count(const hq_network* net, int32_t* launches) {
  if (!net || !launches) return HQ_ERR_INVALID_ARG;
  *launches = net->launches;
  return HQ_OK;
}

hq_status hq_network_destroy(hq_network* net) {
  if (!net) return HQ_ERR_INVALID_ARG;
  for (auto& g : net->graphs) cudaGraphExecDestroy(g.exec);
  for (auto& b : net->buffers) cudaFree(b.base);
  delete net;
  return HQ_OK;
}

hq_status hq_network_check_guards(const hq_network* net, void* stream, int32_t* bad_layer) {
  if (!net) return HQ_ERR_INVALID_ARG;
  if (bad_layer) *bad_layer = -2;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HQ_ERR_CUDA;
  unsigned char band[2 * kGuardBytes];
  for (const auto& b : net->buffers) {
    const unsigned char* base = (const unsigned char*)b.base;
    if (cudaMemcpy(band, base, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess ||
        cudaMemcpy(band + kGuardBytes, base + kGuardBytes + b.bytes, kGuardBytes, cudaMemcpyDeviceToHost) != cudaSuccess)
      return HQ_ERR_CUDA;
    for (size_t k = 0; k < 2 * kGuardBytes; ++k)
      if (band[k] != (unsigned char)kGuardByte) {
        if (bad_layer) *bad_layer = b.layer;
        return HQ_ERR_RANGE;
      }
  }
  return HQ_OK;
}

}  // extern "C"
