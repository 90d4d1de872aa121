// Lowering of convolutions whose channel count does not fit the tensor-core kernel's 32-byte K
// blocks (the 3-channel first layer): the patches of Eq. 3 are written once as rows of a dense
// matrix [pixels][Kp] with Kp = kh*kw*cin rounded up to 32 and zero-filled, the weights likewise
// as [cout][Kp]; the contraction then runs as a 1x1 convolution on the tensor-core kernel.  The
// zero columns add nothing to the INT32 accumulator, so the result is unchanged.
#include "hq_internal.cuh"

namespace {

__global__ void __launch_bounds__(256) patch_matrix_kernel(const unsigned char* __restrict__ in, int n, int h, int w,
                                                           int cin, int kh, int kw, int stride, int pad, int ho, int wo,
                                                           int K, int Kp, uint4* __restrict__ out) {
  const int cpr = Kp >> 4;                                   // 16-byte chunks per output row
  const long long total = (long long)n * ho * wo * cpr;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int j = (int)(i % cpr);
    long long m = i / cpr;
    const int ow = (int)(m % wo); m /= wo;
    const int oh = (int)(m % ho);
    const int img = (int)(m / ho);
    int k = j << 4;
    int tap = k / cin, ci = k - tap * cin;
    int r = tap / kw, s = tap - r * kw;
    unsigned word[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int t = 0; t < 16; ++t, ++k) {
      if (k < K) {
        const int ih = oh * stride + r - pad, iw = ow * stride + s - pad;
        if (ih >= 0 && ih < h && iw >= 0 && iw < w) {
          const unsigned v = __ldg(in + (((long long)img * h + ih) * w + iw) * cin + ci);
          word[t >> 2] |= v << (8 * (t & 3));
        }
        if (++ci == cin) { ci = 0; if (++s == kw) { s = 0; ++r; } }
      }
    }
    out[i] = make_uint4(word[0], word[1], word[2], word[3]);
  }
}

__global__ void pad_weights_kernel(const unsigned char* __restrict__ wgt, int cout, int K, int Kp,
                                   unsigned char* __restrict__ out) {
  const long long total = (long long)cout * Kp;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
       i += (long long)gridDim.x * blockDim.x) {
    const int k = (int)(i % Kp);
    const long long oc = i / Kp;
    out[i] = k < K ? wgt[oc * K + k] : (unsigned char)0;
  }
}

}  // namespace

bool hq_conv_lowering_applies(const ConvArgs& a) {
  if (a.in_bits != 8) return false;
  const long long K = (long long)a.kh * a.kw * a.cin;
  if (K > 4096) return false;                                // meant for thin first layers
  ConvArgs t = a;
  t.cin = (int)((K + 31) / 32 * 32); t.kh = t.kw = 1; t.stride = 1; t.pad = 0; t.h = a.ho; t.w = a.wo;
  return hq_conv_tc_supported(t);
}

size_t hq_conv_lowering_bytes(const ConvArgs& a) {
  const long long Kp = ((long long)a.kh * a.kw * a.cin + 31) / 32 * 32;
  const long long m = (long long)a.n * a.ho * a.wo;
  return (size_t)(((m * Kp + 255) / 256 + ((long long)a.cout * Kp + 255) / 256) * 256);
}

// `scratch` must hold hq_conv_lowering_bytes(a) bytes, 256-byte aligned.
hq_status hq_launch_conv_lowered(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s) {
  const int K = a.kh * a.kw * a.cin;
  const int Kp = (K + 31) / 32 * 32;
  const long long m = (long long)a.n * a.ho * a.wo;
  if (m == 0) return HQ_OK;
  unsigned char* patches = (unsigned char*)scratch;
  unsigned char* wpad = patches + (m * Kp + 255) / 256 * 256;
  {
    const long long total = (long long)a.cout * Kp;
    pad_weights_kernel<<<(int)((total + 255) / 256), 256, 0, s>>>((const unsigned char*)a.wgt, a.cout, K, Kp, wpad);
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  }
  {
    const long long total = m * (Kp >> 4);
    long long blocks = (total + 255) / 256;
    const long long cap = (long long)h->sm_count * 32;
    patch_matrix_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, s>>>(
        (const unsigned char*)a.in, a.n, a.h, a.w, a.cin, a.kh, a.kw, a.stride, a.pad, a.ho, a.wo, K, Kp,
        (uint4*)patches);
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  }
  ConvArgs t = a;
  t.in = patches; t.h = a.ho; t.w = a.wo; t.cin = Kp; t.wgt = wpad; t.kh = t.kw = 1; t.stride = 1; t.pad = 0;
  return hq_launch_conv_tc(h, t, s);
}
