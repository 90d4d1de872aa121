// Windowed sum pooling on wide integers (Appendix E: the pooling branch of an Inception module stays in INT32):
//   out[n, oh, ow, c] = sum over the k x k window of in[n, oh*stride + r - pad, ow*stride + s - pad, c],
// taps outside the image count as 0 and the reciprocal of the window size of an average pool is left to the dyadic
// pair of the consumer (hq_concat_requant, hq_residual_add), so no division touches the data.  Memory bound: a
// thread owns four channels of one output pixel (one 16-byte read per tap of an INT32 tensor, served by L1 / L2 for
// the overlapping windows, one word of an 8-bit tensor) and writes one 16-byte piece of the INT32 output; other
// channel counts and 4-bit inputs read element-wise.
#include "hq_internal.cuh"

namespace {

struct SumPoolArgs {
  const void* in; int32_t* out;
  int32_t n, h, w, ch, bits, is_signed, k, stride, pad, oh_n, ow_n;
  int32_t vec;     // 1: INT32 input with ch % 4 == 0: 16-byte accesses; 2: 8-bit input with ch % 4 == 0: one word per tap
};

// Block x = one output row (image, oh); block y, thread = a piece of that row: (ow, group of four channels), or
// (ow, channel) for element-wise reads.  K = 3 unrolls the window so that its nine reads are in flight together;
// K = 0 takes the window size from the arguments.
template <int K>
__global__ void __launch_bounds__(256) sumpool_kernel(const __grid_constant__ SumPoolArgs a) {
  const int k = K ? K : a.k;
  const int cg = a.vec ? a.ch >> 2 : a.ch;                       // channel groups per pixel
  const int col = blockIdx.y * 256 + threadIdx.x;
  if (col >= a.ow_n * cg) return;
  const int ow = col / cg, g = col - ow * cg;
  const int img = blockIdx.x / a.oh_n, oh = blockIdx.x - img * a.oh_n;
  const int ih0 = oh * a.stride - a.pad, iw0 = ow * a.stride - a.pad;
  const long long o_idx = ((long long)blockIdx.x * a.ow_n + ow) * cg + g;   // in units of the thread's piece
  const long long img_base = (long long)img * a.h * a.w;
  if (a.vec == 1) {
    int4 sum = make_int4(0, 0, 0, 0);
#pragma unroll
    for (int r = 0; r < k; ++r) {
      const int ih = ih0 + r;
#pragma unroll
      for (int s = 0; s < k; ++s) {
        const int iw = iw0 + s;
        if (ih >= 0 && ih < a.h && iw >= 0 && iw < a.w) {
          const int4 v = *((const int4*)((const int*)a.in + (img_base + (long long)ih * a.w + iw) * a.ch) + g);
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
      }
    }
    *((int4*)a.out + o_idx) = sum;
  } else if (a.vec == 2) {
    // 8-bit input: four channels in one 32-bit word per tap, widened as they are added; 16-byte INT32 output
    int4 sum = make_int4(0, 0, 0, 0);
#pragma unroll
    for (int r = 0; r < k; ++r) {
      const int ih = ih0 + r;
#pragma unroll
      for (int s = 0; s < k; ++s) {
        const int iw = iw0 + s;
        if (ih >= 0 && ih < a.h && iw >= 0 && iw < a.w) {
          const unsigned v = __ldg((const unsigned*)a.in + (((img_base + (long long)ih * a.w + iw) * a.ch) >> 2) + g);
          if (a.is_signed) {
            sum.x += (int)(signed char)v; sum.y += (int)(signed char)(v >> 8);
            sum.z += (int)(signed char)(v >> 16); sum.w += (int)v >> 24;
          } else {
            sum.x += (int)(v & 0xFFu); sum.y += (int)((v >> 8) & 0xFFu); sum.z += (int)((v >> 16) & 0xFFu); sum.w += (int)(v >> 24);
          }
        }
      }
    }
    *((int4*)a.out + o_idx) = sum;
  } else {
    int sum = 0;
    for (int r = 0; r < k; ++r) {
      const int ih = ih0 + r;
      if (ih < 0 || ih >= a.h) continue;
      for (int s = 0; s < k; ++s) {
        const int iw = iw0 + s;
        if (iw < 0 || iw >= a.w) continue;
        sum += hq_load_elem(a.in, (img_base + (long long)ih * a.w + iw) * a.ch + g, a.bits, a.is_signed);
      }
    }
    a.out[o_idx] = sum;
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
  a.vec = in->c % 4 != 0 ? 0 : in->bits == 32 ? 1 : in->bits == 8 ? 2 : 0;
  if (a.n == 0) return HQ_OK;
  const long long rows = (long long)a.n * ho, cols = (long long)wo * (a.vec ? a.ch / 4 : a.ch);
  if (rows > 0x7fffffffLL || (cols + 255) / 256 > 65535) return HQ_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)rows, (unsigned)((cols + 255) / 256));
  if (k == 3) sumpool_kernel<3><<<grid, 256, 0, (cudaStream_t)stream>>>(a);
  else sumpool_kernel<0><<<grid, 256, 0, (cudaStream_t)stream>>>(a);
  return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
