// Lowering of convolutions that the direct tensor-core kernel does not take: channel counts that do not
// fit its 32-byte K blocks (the 3-channel first layer), and layers whose activation tensor is too small for
// an im2col-mode tensor map (below 128 KiB).  The patches of Eq. 3 are written once as rows of a dense
// matrix [pixels][Kp] with Kp = kh*kw*cin rounded up to 32 and zero-filled, the weights likewise
// as [cout][Kp]; the contraction then runs as a 1x1 convolution on the tensor-core kernel.  The
// zero columns add nothing to the INT32 accumulator, so the result is unchanged.
#include <mutex>

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

// The same for channel counts that are a multiple of 16 (e.g. the 48-channel branches of an Inception module): the
// window rows, the taps of a filter row and the patch rows are then whole 16-byte pieces, so both passes move
// 16 bytes per access and a patch piece is one shared-memory read.
__global__ void __launch_bounds__(256) patch_matrix_vec16_kernel(const uint4* __restrict__ in, int n, int h, int w,
                                                                 int cin, int kh, int kw, int stride, int pad, int ho, int wo,
                                                                 int K, int Kp, int wseg, int segs, int win_bytes,
                                                                 uint4* __restrict__ out) {
  extern __shared__ uint4 win16[];                           // [kh][win_bytes / 16]
  const int seg = blockIdx.x % segs;
  const int oh = (blockIdx.x / segs) % ho;
  const int img = blockIdx.x / (segs * ho);
  const int ow0 = seg * wseg;
  const int npix = (wo - ow0) < wseg ? (wo - ow0) : wseg;
  const int c16 = cin >> 4, wq = win_bytes >> 4, rowq = w * c16;
  const int col0 = (ow0 * stride - pad) * c16;                // first 16-byte piece of the window inside an input row
  for (int i = threadIdx.x; i < kh * wq; i += blockDim.x) {
    const int r = i / wq, b = i - r * wq;
    const int ih = oh * stride + r - pad, col = col0 + b;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (ih >= 0 && ih < h && col >= 0 && col < rowq) v = __ldg(in + ((long long)img * h + ih) * rowq + col);
    win16[i] = v;
  }
  __syncthreads();
  const int cpr = Kp >> 4, kq = K >> 4, kwq = kw * c16;
  uint4* dst = out + (((long long)img * ho + oh) * wo + ow0) * cpr;
  for (int i = threadIdx.x; i < npix * cpr; i += blockDim.x) {
    const int px = i / cpr, j = i - px * cpr;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (j < kq) {
      const int r = j / kwq, t = j - r * kwq;
      v = win16[r * wq + px * stride * c16 + t];
    }
    dst[i] = v;
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
  if (K > 16384) return false;                               // meant for thin first layers and small late layers
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
    if (a.cin % 16 == 0 && ((uintptr_t)a.in & 15u) == 0 && !a.pitch_w)
      patch_matrix_vec16_kernel<<<(int)blocks, 256, smem, s>>>((const uint4*)a.in, a.n, a.h, a.w, a.cin, a.kh, a.kw,
                                                               a.stride, a.pad, a.ho, a.wo, K, Kp, wseg, segs, win_bytes,
                                                               (uint4*)patches);
    else
    patch_matrix_kernel<<<(int)blocks, 256, smem, s>>>((const unsigned char*)a.in, a.n, a.h, a.w, a.cin, a.kh, a.kw,
                                                       a.stride, a.pad, a.ho, a.wo, K, Kp, wseg, segs, win_bytes,
                                                       (uint4*)patches);
    if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  }
  ConvArgs t = a;
  t.in = patches; t.h = a.ho; t.w = a.wo; t.cin = Kp; t.wgt = wpad; t.kh = t.kw = 1; t.stride = 1; t.pad = 0;
  return hq_launch_conv_tc(h, t, s);
}

// ------------------------------------------------------------------------------------------------
// First layer of ImageNet ResNets (7x7, stride 2, pad 3, 3 input channels) without a patch matrix.
// A space-to-depth copy of the image, s2d[n][y][x][(dy*2+dx)*3 + c] = in[n][2y+dy][2x+dx][c] with the
// 12 values padded to 16 channels, turns the layer into a 4x4 stride-1 convolution with 16-byte
// pixels: output (oh, ow) reads s2d rows oh-2 .. oh+1 (two rows of padding before, one after), and
// weight w2[oc][ty][tx][(dy*2+dx)*3 + c] = w[oc][2ty+dy-1][2tx+dx-1][c] (zero where the 7x7 index falls
// outside 0..6 and in the padded channels).  Zeros add nothing, so the INT32 accumulator is unchanged.
//
// The copy is stored with its zero padding, so the taps of a filter row are contiguous bytes, and the
// tensor-core kernel is handed a 4x1 convolution over "pixels" that are windows of the stored image:
// one window of 8 stored pixels (128 bytes, W pitch 32 bytes: neighbouring windows overlap) feeds TWO
// adjacent outputs, whose 2 x cout values are the window's "output channels": output 2q + o, channel ch is
// virtual channel o*cout + ch of virtual pixel q, i.e. the same byte of the NHWC output tensor read as rows
// of 2*cout bytes.  Virtual channel (o, ch) carries w2[ch][ty][i - o][.] at stored pixel i of the window
// (zero outside 0 <= i - o <= 3).  That gives full 128-byte TMA rows and fills all 128 accumulator lanes
// for cout = 64 (16-byte and 64-byte rows measured 4x and 1.4x slower), at the price of multiplying zeros.
// ------------------------------------------------------------------------------------------------
namespace {

__global__ void __launch_bounds__(256) space_to_depth_kernel(const unsigned char* __restrict__ in, int n, int h, int w,
                                                             uint4* __restrict__ out) {
  // output: [n][h/2 + 3][w/2 + 3] pixels of 16 bytes, the image surrounded by its zero padding (2 before, 1 after).
  // A thread builds two neighbouring output pixels x0 = 2p - 2, x0 + 1: their 2 x 12 source bytes are three aligned
  // words in each of the two image rows (w % 4 == 0 and a 16-byte aligned image make (2 x0) * 3 a multiple of 4).
  const int h2 = h >> 1, w2 = w >> 1, hp = h2 + 3, wp = w2 + 3, pairs = (wp + 1) >> 1;
  const long long total = (long long)n * hp * pairs;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int pr = (int)(i % pairs);
    long long t = i / pairs;
    const int y = (int)(t % hp) - 2;
    const int img = (int)(t / hp);
    const int x0 = 2 * pr - 2;
    unsigned a[4] = {0u, 0u, 0u, 0u}, b[4] = {0u, 0u, 0u, 0u};          // pixels x0 and x0 + 1
    if (y >= 0 && y < h2 && x0 >= 0 && x0 < w2) {                       // w2 is even: x0 + 1 is inside with x0
#pragma unroll
      for (int dy = 0; dy < 2; ++dy) {
        const unsigned* src = (const unsigned*)(in + (((long long)img * h + 2 * y + dy) * w + 2 * x0) * 3);
        const unsigned s0 = __ldg(src), s1 = __ldg(src + 1), s2 = __ldg(src + 2);   // 12 bytes: 6 of pixel x0, 6 of x0 + 1
        // byte k = dy * 6 + j of a 16-byte output pixel
        const unsigned long long pa = (unsigned long long)s0 | ((unsigned long long)(s1 & 0xFFFFu) << 32);       // 6 bytes
        const unsigned long long pb = (unsigned long long)(s1 >> 16) | ((unsigned long long)s2 << 16);           // 6 bytes
        if (dy == 0) { a[0] = (unsigned)pa; a[1] = (unsigned)(pa >> 32); b[0] = (unsigned)pb; b[1] = (unsigned)(pb >> 32); }
        else {
          a[1] |= (unsigned)(pa << 16); a[2] = (unsigned)(pa >> 16);
          b[1] |= (unsigned)(pb << 16); b[2] = (unsigned)(pb >> 16);
        }
      }
    }
    uint4* dst = out + ((long long)img * hp + (y + 2)) * wp + (x0 + 2);
    dst[0] = make_uint4(a[0], a[1], a[2], a[3]);
    if (x0 + 3 < wp) dst[1] = make_uint4(b[0], b[1], b[2], b[3]);
  }
}

// Weights of the 2*cout virtual channels, [2*cout][4 filter rows][128 window bytes], and the per-channel
// constants repeated for both outputs of a window.
__global__ void s2d_weights_kernel(const signed char* __restrict__ w, int cout, signed char* __restrict__ out,
                                   const int32_t* __restrict__ bias, const int32_t* __restrict__ b,
                                   const int32_t* __restrict__ c, int32_t* __restrict__ consts) {
  const int total = 2 * cout * 512;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < total; i += gridDim.x * blockDim.x) {
    const int ch16 = i & 15, px = (i >> 4) & 7, ty = (i >> 7) & 3, v = i >> 9;
    const int o = v / cout, oc = v - o * cout, tx = px - o;
    signed char val = 0;
    if (ch16 < 12 && tx >= 0 && tx < 4) {
      const int cc = ch16 % 3, dx = (ch16 / 3) & 1, dy = ch16 / 6;
      const int r = 2 * ty + dy - 1, sx = 2 * tx + dx - 1;
      if (r >= 0 && r < 7 && sx >= 0 && sx < 7) val = w[((oc * 7 + r) * 7 + sx) * 3 + cc];
    }
    out[i] = val;
    if (i < 2 * cout) {
      const int ch = i % cout;
      consts[i] = bias ? bias[ch] : 0;
      consts[2 * cout + i] = b ? b[ch] : 0;
      consts[4 * cout + i] = c ? c[ch] : 1;
    }
  }
}

// scratch layout: padded image | virtual weights | bias, b, c of the virtual channels
struct S2dLayout { long long img_bytes, wts_off, wts_bytes, consts_off, total; };
S2dLayout s2d_layout(const ConvArgs& a) {
  S2dLayout l;
  l.img_bytes = (long long)a.n * (a.h / 2 + 3) * (a.w / 2 + 3) * 16;
  l.wts_off = (l.img_bytes + 255) / 256 * 256;          // the last window reads 48 bytes past the image: into the weights
  l.wts_bytes = (long long)2 * a.cout * 512;
  l.consts_off = l.wts_off + (l.wts_bytes + 255) / 256 * 256;
  l.total = l.consts_off + ((long long)6 * a.cout * 4 + 255) / 256 * 256;
  return l;
}

ConvArgs s2d_conv_args(const ConvArgs& a, const void* scratch) {
  ConvArgs t = a;
  const S2dLayout l = s2d_layout(a);
  const int h2 = a.h / 2, w2 = a.w / 2, hp = h2 + 3, wp = w2 + 3;
  const unsigned char* base = (const unsigned char*)scratch;
  // weights and constants of the virtual channels: prepared once by the caller (a network), else in the scratch block
  const unsigned char* prep = a.wgt_widened ? (const unsigned char*)a.wgt_widened : base + l.wts_off;
  const int32_t* consts = (const int32_t*)(prep + (l.consts_off - l.wts_off));
  t.wgt_widened = nullptr;
  t.in = base; t.wgt = prep;
  t.h = hp; t.w = w2 / 2; t.cin = 128; t.kh = 4; t.kw = 1; t.stride = 1; t.pad = 0; t.pad_after_delta = 0;
  t.pitch_w = 32; t.pitch_h = (long long)wp * 16; t.pitch_n = (long long)hp * wp * 16;
  t.cout = 2 * a.cout; t.wo = a.wo / 2;
  t.bias = consts; t.b = consts + 2 * a.cout; t.c = consts + 4 * a.cout;
  return t;
}
}  // namespace

bool hq_conv_s2d_applies(const ConvArgs& a) {
  if (a.in_bits != 8 || a.cin != 3 || a.kh != 7 || a.kw != 7 || a.stride != 2 || a.pad != 3) return false;
  if ((a.h & 1) || (a.w & 3) || a.pitch_w || a.res || a.out_bits != 8) return false;       // pairs of outputs: w/2 even
  if ((long long)a.cout * 1024 >= (1ll << 31)) return false;
  const ConvArgs t = s2d_conv_args(a, a.in);
  return hq_conv_tc_supported(t) && !hq_conv_tc_small_im2col(t);   // small images take the patch-matrix form
}

size_t hq_conv_s2d_bytes(const ConvArgs& a) { return (size_t)s2d_layout(a).total; }

// The layer's weights in the form of the virtual channels, with their constants: a network prepares them once when it
// is built and hands the block over as ConvArgs::wgt_widened; `buf` holds hq_conv_s2d_prepared_bytes(a) bytes.
size_t hq_conv_s2d_prepared_bytes(const ConvArgs& a) { const S2dLayout l = s2d_layout(a); return (size_t)(l.total - l.wts_off); }
cudaError_t hq_prepare_conv_s2d(const ConvArgs& a, void* buf, cudaStream_t s) {
  const S2dLayout l = s2d_layout(a);
  s2d_weights_kernel<<<(2 * a.cout * 512 + 255) / 256, 256, 0, s>>>((const signed char*)a.wgt, a.cout, (signed char*)buf, a.bias, a.b, a.c,
                                                                   (int32_t*)((unsigned char*)buf + (l.consts_off - l.wts_off)));
  return cudaGetLastError();
}

// `scratch` must hold hq_conv_s2d_bytes(a) bytes, 256-byte aligned.
hq_status hq_launch_conv_s2d(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s) {
  if (a.n == 0) return HQ_OK;
  const S2dLayout l = s2d_layout(a);
  unsigned char* base = (unsigned char*)scratch;
  if (!a.wgt_widened && hq_prepare_conv_s2d(a, base + l.wts_off, s) != cudaSuccess) return HQ_ERR_CUDA;
  const long long px = l.img_bytes / 16 / 2;          // a thread builds two pixels
  long long blocks = (px + 255) / 256;
  const long long cap = (long long)h->sm_count * 32;
  space_to_depth_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, s>>>((const unsigned char*)a.in, a.n, a.h, a.w, (uint4*)base);
  if (cudaGetLastError() != cudaSuccess) return HQ_ERR_CUDA;
  return hq_launch_conv_tc(h, s2d_conv_args(a, scratch), s);
}

// ------------------------------------------------------------------------------------------------
// 4-bit operands on the tensor-core kernel.  sm_100 has no 4-bit integer MMA, so packed INT4
// activations and weights (two per byte, even element in the low nibble) are widened to one byte
// per value and the contraction of Eq. 3 runs on the 8-bit kernel; the integers, hence the results,
// are unchanged.  This version widens in global memory (a scratch copy of the layer input and of
// the weights) ahead of the convolution.
// ------------------------------------------------------------------------------------------------
namespace {

template <bool SIGNED>
__device__ __forceinline__ uint4 widen4_vec(uint2 v) {
  unsigned o[4];
  const unsigned w[2] = {v.x, v.y};
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    unsigned lo = w[k] & 0x0F0F0F0Fu, hi = (w[k] >> 4) & 0x0F0F0F0Fu;
    if (SIGNED) { lo |= (lo & 0x08080808u) * 0x1Eu; hi |= (hi & 0x08080808u) * 0x1Eu; }   // sign-extend each nibble
    o[2 * k] = __byte_perm(lo, hi, 0x5140);          // n0 n1 n2 n3
    o[2 * k + 1] = __byte_perm(lo, hi, 0x7362);      // n4 n5 n6 n7
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// 8 packed bytes -> 16 bytes; element 2j = low nibble of byte j.  Four independent loads per thread and trip.
template <bool SIGNED>
__global__ void __launch_bounds__(256) widen4_kernel(const uint2* __restrict__ in, long long n_vec, uint4* __restrict__ out) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < n_vec; i += 4 * stride) {
    uint2 v[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) v[u] = __ldg(in + i + u * stride);
#pragma unroll
    for (int u = 0; u < 4; ++u) out[i + u * stride] = widen4_vec<SIGNED>(v[u]);
  }
  for (; i < n_vec; i += stride) out[i] = widen4_vec<SIGNED>(__ldg(in + i));
}

// One byte per value -> two values per byte (low nibble first); 8 bytes in, 4 bytes out per thread and step.
__global__ void __launch_bounds__(256) pack4_kernel(const uint2* __restrict__ in, long long n_vec, unsigned* __restrict__ out) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
    const uint2 v = __ldg(in + i);
    const unsigned lo = (v.x & 0x0F0F0F0Fu) | ((v.x >> 4) & 0x00F000F0u);      // bytes 0 and 2 hold the packed pairs
    const unsigned hi = (v.y & 0x0F0F0F0Fu) | ((v.y >> 4) & 0x00F000F0u);
    out[i] = __byte_perm(lo, hi, 0x6420);
  }
}

cudaError_t launch_widen4(const void* in, long long elems, int is_signed, void* out, int sm_count, cudaStream_t s) {
  const long long n_vec = elems / 16;                  // callers guarantee a multiple of 16 elements
  if (n_vec == 0) return cudaSuccess;
  long long blocks = (n_vec + 255) / 256;
  const long long cap = (long long)sm_count * 16;
  const int grid = (int)(blocks < cap ? blocks : cap);
  if (is_signed) widen4_kernel<true><<<grid, 256, 0, s>>>((const uint2*)in, n_vec, (uint4*)out);
  else widen4_kernel<false><<<grid, 256, 0, s>>>((const uint2*)in, n_vec, (uint4*)out);
  return cudaGetLastError();
}

}  // namespace

bool hq_conv_widen4_applies(const ConvArgs& a) {
  // (16 values per step of the widening kernels; channel counts the direct kernel does not take go on to the
  // patch-matrix form after widening, e.g. the 48-channel 5x5 branch of an Inception module)
  if (a.in_bits != 4) return false;
  if (((long long)a.n * a.h * a.w * a.cin) % 16 != 0 || ((long long)a.cout * a.kh * a.kw * a.cin) % 16 != 0) return false;
  ConvArgs t = a;
  t.in_bits = 8;
  return hq_conv_tc_supported(t) || hq_conv_lowering_applies(t);
}

static size_t widen4_copy_bytes(const ConvArgs& a) {
  const long long x = (long long)a.n * a.h * a.w * a.cin, w = (long long)a.cout * a.kh * a.kw * a.cin;
  return (size_t)(((x + 255) / 256 + (w + 255) / 256) * 256);
}

// the widened copies, plus the patch matrix when the widened layer is one the direct kernel declines
size_t hq_conv_widen4_bytes(const ConvArgs& a) {
  ConvArgs t = a;
  t.in_bits = 8;
  const bool lowered = (!hq_conv_tc_supported(t) || hq_conv_tc_small_im2col(t)) && hq_conv_lowering_applies(t);
  return widen4_copy_bytes(a) + (lowered ? hq_conv_lowering_bytes(t) : 0);
}

// `scratch` must hold hq_conv_widen4_bytes(a) bytes, 256-byte aligned.
hq_status hq_launch_conv_widen4(hq_handle* h, const ConvArgs& a, void* scratch, cudaStream_t s) {
  const long long x = (long long)a.n * a.h * a.w * a.cin, w = (long long)a.cout * a.kh * a.kw * a.cin;
  unsigned char* xw = (unsigned char*)scratch;
  unsigned char* ww = xw + (x + 255) / 256 * 256;
  // (weights first: the convolution fetches resident weights without waiting for the launch just before it)
  if (!a.wgt_widened && launch_widen4(a.wgt, w, 1, ww, h->sm_count, s) != cudaSuccess) return HQ_ERR_CUDA;
  if (launch_widen4(a.in, x, a.in_signed, xw, h->sm_count, s) != cudaSuccess) return HQ_ERR_CUDA;
  ConvArgs t = a;
  t.in = xw; t.wgt = a.wgt_widened ? a.wgt_widened : ww; t.in_bits = 8;
  const hq_status st = hq_launch_conv_tc(h, t, s);
  if (st != HQ_ERR_UNSUPPORTED || !hq_conv_lowering_applies(t)) return st;
  return hq_launch_conv_lowered(h, t, xw + widen4_copy_bytes(a), s);      // declined by the direct kernel: patch matrix
}

cudaError_t hq_launch_pack4(const void* in, long long values, void* out, int sm_count, cudaStream_t s) {
  const long long n_vec = values / 8;                  // callers guarantee a multiple of 8 values
  if (n_vec == 0) return cudaSuccess;
  const long long blocks = (n_vec + 255) / 256, cap = (long long)sm_count * 16;
  pack4_kernel<<<(int)(blocks < cap ? blocks : cap), 256, 0, s>>>((const uint2*)in, n_vec, (unsigned*)out);
  return cudaGetLastError();
}

cudaError_t hq_launch_widen_weights(const void* wgt, long long values, void* out, int sm_count, cudaStream_t s) {
  return launch_widen4(wgt, values, 1, out, sm_count, s);
}

// ------------------------------------------------------------------------------------------------
// hq_conv2d_noalloc: the lowered convolution for callers that may not allocate device memory.
//
// The patch matrix and the padded weights, which hq_conv2d keeps in a buffer it allocates, live here
// in a fixed array inside the library's own device image.  Every GPU that loads the library carries
// the array until the process exits, so it is kept modest: HQ_NOALLOC_SCRATCH_BYTES.
// ------------------------------------------------------------------------------------------------
#define HQ_NOALLOC_SCRATCH_BYTES (8u << 20)      /* 8 MiB: e.g. one 224x224x3 image through a 7x7/2 first layer needs 2 MiB */

static __device__ __align__(256) unsigned char g_noalloc_scratch[HQ_NOALLOC_SCRATCH_BYTES];
static __device__ uint32_t g_noalloc_status;     // written by a kernel whose bounded wait ran out

namespace {

// Host-side record per device ordinal.  The array names above are only host-side stand-ins for the
// device objects; the addresses the kernels need come from cudaGetSymbolAddress, taken once per
// device while that device is current.
struct NoAllocDevice { bool ready; void* scratch; uint32_t* status; int sm_count; };
constexpr int kMaxDevices = 64;
NoAllocDevice g_noalloc_dev[kMaxDevices];
std::mutex g_noalloc_mutex;     // first calls from several host threads: one of them fills the record, the others wait

hq_status noalloc_setup(int dev) {
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  NoAllocDevice& d = g_noalloc_dev[dev];
  if (d.ready) return HQ_OK;
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return HQ_ERR_CUDA;
  if (major != 10) return HQ_ERR_UNSUPPORTED;                  // kernels are built for sm_100a only
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return HQ_ERR_CUDA;
  if (!hq_conv_tc_init()) return HQ_ERR_CUDA;                  // driver entry points, shared-memory limit
  void* scratch = nullptr;
  void* status = nullptr;
  if (cudaGetSymbolAddress(&scratch, g_noalloc_scratch) != cudaSuccess || !scratch) return HQ_ERR_CUDA;
  if (cudaGetSymbolAddress(&status, g_noalloc_status) != cudaSuccess || !status) return HQ_ERR_CUDA;
  d.scratch = scratch; d.status = (uint32_t*)status; d.sm_count = sms; d.ready = true;
  return HQ_OK;
}

inline bool na_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" hq_status hq_conv2d_noalloc(const hq_tensor* in, const hq_conv_desc* d, hq_tensor* out, void* stream) {
  if (!in || !d || !out || !in->data || !out->data || !d->w) return HQ_ERR_INVALID_ARG;
  if (in->bits != 8 || d->w_bits != 8) return HQ_ERR_UNSUPPORTED;          // 8-bit operands only
  if (!(out->bits == 8 || out->bits == 4 || out->bits == 32)) return HQ_ERR_INVALID_ARG;
  if (in->n < 0 || in->h < 1 || in->w < 1 || in->c < 1) return HQ_ERR_INVALID_ARG;
  if (d->kh < 1 || d->kw < 1 || d->stride < 1 || d->pad < 0 || d->cout < 1 || d->cin != in->c) return HQ_ERR_INVALID_ARG;
  if (in->h + 2 * d->pad < d->kh || in->w + 2 * d->pad < d->kw) return HQ_ERR_INVALID_ARG;
  const int ho = (in->h + 2 * d->pad - d->kh) / d->stride + 1, wo = (in->w + 2 * d->pad - d->kw) / d->stride + 1;
  if (out->n != in->n || out->h != ho || out->w != wo || out->c != d->cout) return HQ_ERR_INVALID_ARG;
  if (out->bits == 4 && (d->cout & 1)) return HQ_ERR_INVALID_ARG;
  if (!na_aligned16(in->data) || !na_aligned16(out->data) || !na_aligned16(d->w)) return HQ_ERR_ALIGNMENT;
  ConvArgs a{};
  a.in = in->data; a.n = in->n; a.h = in->h; a.w = in->w; a.cin = in->c; a.in_bits = 8; a.in_signed = in->is_signed;
  a.wgt = d->w; a.cout = d->cout; a.kh = d->kh; a.kw = d->kw; a.stride = d->stride; a.pad = d->pad;
  a.bias = d->bias; a.b = d->requant.b; a.c = d->requant.c;
  a.relu = d->relu; a.qmin = d->qmin; a.qmax = d->qmax;
  a.out = out->data; a.ho = ho; a.wo = wo; a.out_bits = out->bits; a.out_signed = out->is_signed;
  if (out->bits == 32) {
    if (d->residual) return HQ_ERR_INVALID_ARG;
  } else {
    if (!d->requant.b || !d->requant.c) return HQ_ERR_INVALID_ARG;
    long long lo = out->is_signed ? -(1LL << (out->bits - 1)) : 0;
    long long hi = out->is_signed ? (1LL << (out->bits - 1)) - 1 : (1LL << out->bits) - 1;
    if (d->qmin > d->qmax || d->qmin < lo || d->qmax > hi) return HQ_ERR_INVALID_ARG;
    if (d->residual) {
      const hq_tensor* r = d->residual;
      if (!r->data || !(r->bits == 8 || r->bits == 32) || r->n != out->n || r->h != ho || r->w != wo || r->c != d->cout ||
          !d->res_rescale.b || !d->res_rescale.c) return HQ_ERR_INVALID_ARG;
      if (!na_aligned16(r->data)) return HQ_ERR_ALIGNMENT;
      a.res = r->data; a.res_bits = r->bits; a.res_signed = r->is_signed; a.rb = d->res_rescale.b; a.rc = d->res_rescale.c;
    }
  }
  if ((long long)d->kh * d->kw * d->cin > 4096 || !hq_conv_lowering_applies(a)) return HQ_ERR_UNSUPPORTED;
  if (hq_conv_lowering_bytes(a) > (size_t)HQ_NOALLOC_SCRATCH_BYTES) return HQ_ERR_WORKSPACE;   // beyond the fixed array

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return HQ_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return HQ_ERR_UNSUPPORTED;
  const hq_status st = noalloc_setup(dev);       // first call on this device only
  if (st != HQ_OK) return st;
  const NoAllocDevice& nd = g_noalloc_dev[dev];
  cudaStream_t s = (cudaStream_t)stream;
  // The array keeps whatever the last call left.  The patch matrix and the padded weights are
  // rewritten in full (zero columns included) before anything reads them; only the status word
  // has to start at zero.
  if (cudaMemsetAsync(nd.status, 0, sizeof(uint32_t), s) != cudaSuccess) return HQ_ERR_CUDA;
  hq_handle tmp{};
  tmp.device = dev; tmp.conv_path = 0; tmp.sm_count = nd.sm_count; tmp.dev_status = nd.status;
  tmp.workspace = nullptr; tmp.workspace_bytes = 0;
  return hq_launch_conv_lowered(&tmp, a, nd.scratch, s);
}

// Wait for `stream` and report an expired device-side wait of the hq_conv2d_noalloc calls queued on it.
extern "C" hq_status hq_conv2d_noalloc_sync(void* stream) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return HQ_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return HQ_ERR_UNSUPPORTED;
  const hq_status st = noalloc_setup(dev);
  if (st != HQ_OK) return st;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return HQ_ERR_CUDA;
  uint32_t word = 0;
  if (cudaMemcpy(&word, g_noalloc_dev[dev].status, sizeof(word), cudaMemcpyDeviceToHost) != cudaSuccess) return HQ_ERR_CUDA;
  return word != 0 ? HQ_ERR_TIMEOUT : HQ_OK;
}
