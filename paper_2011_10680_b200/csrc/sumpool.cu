// Windowed sum pooling on wide integers (Appendix E: the pooling branch of an Inception module stays in INT32):
//   out[n, oh, ow, c] = sum over the k x k window of in[n, oh*stride + r - pad, ow*stride + s - pad, c],
// taps outside the image count as 0 and the reciprocal of the window size of an average pool is left to the dyadic
// pair of the consumer (hq_concat_requant, hq_residual_add), so no division touches the data.  Memory bound: a
// thread owns four channels of one output pixel (one 16-byte read per tap of an INT32 tensor, served by L1 / L2 for
// the overlapping windows, one word of an 8-bit tensor) and writes one 16-byte piece of the INT32 output; other
// channel counts and 4-bit inputs read element-wise.  The 3 x 3 / stride 1 / pad 1 window of the Inception modules has
// its own kernel, which forms every row's three-pixel sum once (sumpool3_rows_kernel).
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

// 3 x 3 / stride 1 / pad 1 (the pooling branch of an Inception module) with four channels per thread.  A thread walks
// down one output column of a strip of rows: the sum over the three pixels (ow - 1, ow, ow + 1) of an input row is
// formed once and serves the three output rows it belongs to, so an output costs three reads instead of nine; the
// sums of the last two rows stay in registers.  Consecutive threads hold consecutive channel groups of a pixel, then
// the next pixel: reads and the 16-byte stores are consecutive across a warp.  8-bit inputs are summed as two pairs
// of 16-bit lanes per word (nine bytes add up to at most 2295); signed bytes are biased by 128 first (a tap outside
// the image counts as the biased zero), and 9 * 128 comes off at the end.
template <int IN8, int SIGNED>
__global__ void __launch_bounds__(256) sumpool3_rows_kernel(const __grid_constant__ SumPoolArgs a, int strip_rows, int strips) {
  const int cg = a.ch >> 2;
  const int col = blockIdx.x * 256 + threadIdx.x;
  if (col >= a.w * cg) return;
  const int ow = col / cg, g = col - ow * cg;
  const int img = blockIdx.y / strips, strip = blockIdx.y - img * strips;
  const int r0 = strip * strip_rows, r1 = min(r0 + strip_rows, a.h);
  const bool left = ow > 0, right = ow + 1 < a.w;
  const long long img_row0 = (long long)img * a.h;
  int4* __restrict__ outp = (int4*)a.out + ((img_row0 + r0) * a.w + ow) * cg + g;
  const long long out_step = (long long)a.w * cg;
  if constexpr (IN8) {
    const unsigned* __restrict__ in = (const unsigned*)a.in;
    constexpr unsigned kBias = SIGNED ? 0x80808080u : 0u;
    // the row's three-pixel sum as (bytes 0, 2) and (bytes 1, 3) in 16-bit lanes
    auto hsum = [&](int ih, unsigned& lo, unsigned& hi) {
      unsigned v0 = 0, v1 = 0, v2 = 0;
      if (ih >= 0 && ih < a.h) {
        const unsigned* row = in + ((img_row0 + ih) * a.w + ow) * cg + g;
        v1 = __ldg(row);
        if (left) v0 = __ldg(row - cg);
        if (right) v2 = __ldg(row + cg);
      }
      v0 ^= kBias; v1 ^= kBias; v2 ^= kBias;
      lo = (v0 & 0x00FF00FFu) + (v1 & 0x00FF00FFu) + (v2 & 0x00FF00FFu);
      hi = ((v0 >> 8) & 0x00FF00FFu) + ((v1 >> 8) & 0x00FF00FFu) + ((v2 >> 8) & 0x00FF00FFu);
    };
    unsigned l0, h0, l1, h1;
    hsum(r0 - 1, l0, h0);
    hsum(r0, l1, h1);
#pragma unroll 4
    for (int oh = r0; oh < r1; ++oh, outp += out_step) {
      unsigned l2, h2;
      hsum(oh + 1, l2, h2);
      const unsigned lo = l0 + l1 + l2, hi = h0 + h1 + h2;
      constexpr int kOff = SIGNED ? 9 * 128 : 0;
      *outp = make_int4((int)(lo & 0xFFFFu) - kOff, (int)(hi & 0xFFFFu) - kOff, (int)(lo >> 16) - kOff, (int)(hi >> 16) - kOff);
      l0 = l1; h0 = h1; l1 = l2; h1 = h2;
    }
  } else {
    const int4* __restrict__ in = (const int4*)a.in;
    auto hsum = [&](int ih) -> int4 {
      int4 s = make_int4(0, 0, 0, 0);
      if (ih >= 0 && ih < a.h) {
        const int4* row = in + ((img_row0 + ih) * a.w + ow) * cg + g;
        s = __ldg(row);
        if (left) { const int4 v = __ldg(row - cg); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
        if (right) { const int4 v = __ldg(row + cg); s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w; }
      }
      return s;
    };
    int4 s0 = hsum(r0 - 1), s1 = hsum(r0);
#pragma unroll 4
    for (int oh = r0; oh < r1; ++oh, outp += out_step) {
      const int4 s2 = hsum(oh + 1);
      *outp = make_int4(s0.x + s1.x + s2.x, s0.y + s1.y + s2.y, s0.z + s1.z + s2.z, s0.w + s1.w + s2.w);
      s0 = s1; s1 = s2;
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
  a.vec = in->c % 4 != 0 ? 0 : in->bits == 32 ? 1 : in->bits == 8 ? 2 : 0;
  if (a.n == 0) return HQ_OK;
  if (a.vec && k == 3 && stride == 1 && pad == 1) {
    // strips of rows: long enough that the two extra input rows per strip matter little, short enough to fill the GPU
    const long long cols3 = (long long)a.w * (a.ch / 4);
    int strip_rows = 8;
    while (strip_rows > 2 && (cols3 + 255) / 256 * a.n * ((a.h + strip_rows - 1) / strip_rows) < 16LL * h->sm_count) strip_rows >>= 1;
    const int strips = (a.h + strip_rows - 1) / strip_rows;
    if ((cols3 + 255) / 256 <= 0x7fffffffLL && (long long)a.n * strips <= 65535) {
      const dim3 grid3((unsigned)((cols3 + 255) / 256), (unsigned)(a.n * strips));
      cudaStream_t st = (cudaStream_t)stream;
      if (a.vec == 1) sumpool3_rows_kernel<0, 0><<<grid3, 256, 0, st>>>(a, strip_rows, strips);
      else if (a.is_signed) sumpool3_rows_kernel<1, 1><<<grid3, 256, 0, st>>>(a, strip_rows, strips);
      else sumpool3_rows_kernel<1, 0><<<grid3, 256, 0, st>>>(a, strip_rows, strips);
      return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
    }
  }
  const long long rows = (long long)a.n * ho, cols = (long long)wo * (a.vec ? a.ch / 4 : a.ch);
  if (rows > 0x7fffffffLL || (cols + 255) / 256 > 65535) return HQ_ERR_UNSUPPORTED;
  const dim3 grid((unsigned)rows, (unsigned)((cols + 255) / 256));
  if (k == 3) sumpool_kernel<3><<<grid, 256, 0, (cudaStream_t)stream>>>(a);
  else sumpool_kernel<0><<<grid, 256, 0, (cudaStream_t)stream>>>(a);
  return cudaGetLastError() == cudaSuccess ? HQ_OK : HQ_ERR_CUDA;
}
