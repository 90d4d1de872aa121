// Windowed sum pooling on wide integers (Appendix E: the pooling branch of an Inception module stays in INT32):
//   out[n, oh, ow, c] = sum over the k x k window of in[n, oh*stride + r - pad, ow*stride + s - pad, c],
// taps outside the image count as 0 and the reciprocal of the window size of an average pool is left to the dyadic
// pair of the consumer (hq_concat_requant, hq_residual_add), so no division touches the data.  Memory bound: a
// thread owns four channels of one output pixel (one 16-byte read per tap of an INT32 tensor, served by L1 / L2 for
// the overlapping windows) and writes one 16-byte piece of the INT32 output; other channel counts and 8-/4-bit
// inputs read element-wise.
#include "hq_internal.cuh"

namespace {

struct SumPoolArgs {
  const void* in; int32_t* out;
  int32_t n, h, w, ch, bits, is_signed, k, stride, pad, oh_n, ow_n;
  int32_t vec;     // 1: INT32 input with ch % 4 == 0: 16-byte accesses
};

__global__ void __launch_bounds__(256) sumpool_kernel(const __grid_constant__ SumPoolArgs a) {
  const int cg = a.vec ? a.ch >> 2 : a.ch;                       // channel groups per pixel
  const long long total = (long long)a.n * a.oh_n * a.ow_n * cg;
  for (long long t = (long long)blockIdx.x * 256 + threadIdx.x; t < total; t += (long long)gridDim.x * 256) {
    const int g = (int)(t % cg);
    long long pix = t / cg;
    const int ow = (int)(pix % a.ow_n); pix /= a.ow_n;
    const int oh = (int)(pix % a.oh_n);
    const long long img = pix / a.oh_n;
    const int ih0 = oh * a.stride - a.pad, iw0 = ow * a.stride - a.pad;
    if (a.vec) {
      int4 sum = make_int4(0, 0, 0, 0);
      for (int r = 0; r < a.k; ++r) {
        const int ih = ih0 + r;
        if (ih < 0 || ih >= a.h) continue;
        for (int s = 0; s < a.k; ++s) {
          const int iw = iw0 + s;
          if (iw < 0 || iw >= a.w) continue;
          const int4 v = *((const int4*)((const int*)a.in + ((img * a.h + ih) * a.w + iw) * a.ch) + g);
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
      }
      *((int4*)(a.out + t * 4)) = sum;                             // t enumerates the output's 16-byte pieces in order
    } else {
      int sum = 0;
      for (int r = 0; r < a.k; ++r) {
        const int ih = ih0 + r;
        if (ih < 0 || ih >= a.h) continue;
        for (int s = 0; s < a.k; ++s) {
          const int iw = iw0 + s;
          if (iw < 0 || iw >= a.w) continue;
          sum += hq_load_elem(a.in, ((img * a.h + ih) * a.w + iw) * a.ch + g, a.bits, a.is_signed);
        }
      }
      a.out[t] = sum;
    }
  }
}

}  // namespace

extern "C" hq_status hq_sumpool(hq_handle* h, const hq_tensor* in, int32_t k, int32_t stride, int32_t pad,
                                hq_tensor* out, void* stream) {
  if (!h || !in || !out || !in->data || !out->data) return HQ_ERR_INVALID_ARG;
  if (in->bits != 4 && in->bits != 8 && in->bits != 32) return HQ_ERR_INVALID_ARG;
  if (in->n < 0 || in->h < 1 || in->w < 1 || in->c < 1 || (in->bits == 4 && (in->c & 1))) return HQ_ERR_INVALID_ARG;
  if (k < 1 || stride < 1 || pad < 0 || pad >= k) return HQ_ERR_INVALID_ARG;
  if (in->h + 2 * pad < k || in->w + 2 * pad < k) return HQ_ERR_INVALID_ARG;
  const int ho = (in->h + 2 * pad - k) / stride + 1, wo = (in->w + 2 * pad - k) / stride + 1;
  if (out->bits != 32 || out->n != in->n || out->h != ho || out->w != wo || out->c != in->c) return HQ_ERR_INVALID_ARG;
  if (((uintptr_t)in->data & 15u) || ((uintptr_t)out->data & 15u)) return HQ_ERR_ALIGNMENT;
  if ((long long)k * k > (1LL << 23) && in->bits != 32) return HQ_ERR_UNSUPPORTED;
  SumPoolArgs a{};
  a.in = in->data; a.out = (int32_t*)out->data;
  a.n = in->n; a.h = in->h; a.w = in->w; a.ch = in->c; a.bits = in->bits; a.is_signed = in->bits == 32 ? 1 : in->is_signed;
  a.k = k; a.stride = stride; a.pad = pad; a.oh_n = ho; a.ow_n = wo;
  a.vec = (in->bits == 32 && in->c % 4 == 0) ? 1 : 0;
  const long long total = (long long)a.n * ho * wo * (a.vec ? a.ch / 4 : a.ch);
  if (total == 0) return HQ_OK;
  long long blocks = (total + 255) / 256;
  const long long cap = (long long)h->sm_count * 32;
  if (blocks > cap) blocks = cap;
  sumpool_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(a);
  return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
