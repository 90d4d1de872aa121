// Lowering of convolutions whose channel count does not fit the tensor-core kernel's 32-byte K
// blocks (the 3-channel first layer): the patches of Eq. 3 are written once as rows of a dense
// matrix [pixels][Kp] with Kp = kh*kw*cin rounded up to 32 and zero-filled, the weights likewise
// as [cout][Kp]; the contraction then runs as a 1x1 convolution on the tensor-core kernel.  The
// zero columns add nothing to the INT32 accumulator, so the result is unchanged.
#include "hq_internal.cuh"

namespace {

// One block builds the patch rows of `wseg` consecutive output pixels of one output row.  The kh
// input rows those pixels touch are first copied into shared memory (zero outside the image), so
// that every output byte is one shared-memory read: for a fixed filter row the (kw, cin) taps of a
// pixel are contiguous in NHWC, hence patch byte k = r*(kw*cin) + t sits at window byte
// (ow_local*stride*cin + t) of window row r.
__global__ void __launch_bounds__(256) patch_matrix_kernel(const unsigned char* __restrict__ in, int n, int h, int w,
                                                           int cin, int kh, int kw, int stride, int pad, int ho, int wo,
                                                           int K, int Kp, int wseg, int segs, int win_bytes,
                                                           uint4* __restrict__ out) {
  extern __shared__ unsigned char win[];                     // [kh][win_bytes]
  const int seg = blockIdx.x % segs;
  const int oh = (blockIdx.x / segs) % ho;
  const int img = blockIdx.x / (segs * ho);
  const int ow0 = seg * wseg;
  const int npix = (wo - ow0) < wseg ? (wo - ow0) : wseg;
  const int col0 = (ow0 * stride - pad) * cin;                // byte offset of the window inside an input row
  const int row_bytes = w * cin;
  for (int i = threadIdx.x; i < kh * win_bytes; i += blockDim.x) {
    const int r = i / win_bytes, b = i - r * win_bytes;
    const int ih = oh * stride + r - pad, col = col0 + b;
    unsigned char v = 0;
    if (ih >= 0 && ih < h && col >= 0 && col < row_bytes) v = __ldg(in + ((long long)img * h + ih) * row_bytes + col);
    win[i] = v;
  }
  __syncthreads();
  const int cpr = Kp >> 4, kwc = kw * cin;
  uint4* dst = out + (((long long)img * ho + oh) * wo + ow0) * cpr;
  for (int i = threadIdx.x; i < npix * cpr; i += blockDim.x) {
    const int px = i / cpr, j = i - px * cpr;
    int k = j << 4;
    int r = k / kwc, t = k - r * kwc;
    const unsigned char* src = win + px * stride * cin;
    unsigned word[4] = {0u, 0u, 0u, 0u};
#pragma unroll
    for (int e = 0; e < 16; ++e, ++k) {
      if (k < K) {
        word[e >> 2] |= (unsigned)src[r * win_bytes + t] << (8 * (e & 3));
        if (++t == kwc) { t = 0; ++r; }
      }
    }
    dst[i] = make_uint4(word[0], word[1], word[2], word[3]);
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
  const int wseg = a.wo < 64 ? a.wo : 64;
  if ((long long)a.kh * ((wseg - 1) * a.stride + a.kw) * a.cin > 48 * 1024) return false;   // window must fit shared memory
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
    int wseg = a.wo < 64 ? a.wo : 64;
    const int win_bytes = ((wseg - 1) * a.stride + a.kw) * a.cin;
    const int segs = (a.wo + wseg - 1) / wseg;
    const size_t smem = (size_t)a.kh * win_bytes;
    if (smem > 48 * 1024) return HQ_ERR_UNSUPPORTED;
    const long long blocks = (long long)a.n * a.ho * segs;
    if (blocks >= (1ll << 31)) return HQ_ERR_UNSUPPORTED;
    patch_matrix_kernel<<<(int)blocks, 256, smem, s>>>((const unsigned char*)a.in, a.n, a.h, a.w, a.cin, a.kh, a.kw,
                                                       a.stride, a.pad, a.ho, a.wo, K, Kp, wseg, segs, win_bytes,
                                                       (uint4*)patches);
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  }
  ConvArgs t = a;
  t.in = patches; t.h = a.ho; t.w = a.wo; t.cin = Kp; t.wgt = wpad; t.kh = t.kw = 1; t.stride = 1; t.pad = 0;
  return hq_launch_conv_tc(h, t, s);
}
