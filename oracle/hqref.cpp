// CPU oracle for HAWQ-V3 integer-only inference arithmetic.
//
// TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition that the CUDA library is
// compared against.  It shares no code, header, table or helper with the CUDA library, and only
// the tests, the smoke check and the benchmark's cpu_baseline leg may load it.
//
// Everything here is integer arithmetic: there is no floating-point type and no division in this
// translation unit (the paper's claim for the inference pipeline, Section 1 and Appendix H).
//
//   * contraction q_w * q_h with wide accumulation ............ Eq. 3 (Section 3.1)
//   * INT32 bias of the folded BN added to the accumulator ..... Section 3.2, Appendix D
//   * dyadic requantization  q_a = Int((b / 2^c) * acc) ........ Eq. 4 and the DN(.) definition
//   * residual add, each branch rescaled and rounded, then added  Section 3.3, Appendix G
//   * pooling on wide integers ................................. Appendix E
//
// Readings of points the paper leaves open (all also listed in the design notes):
//   Int(.) is round-half-up, written as add-half-then-arithmetic-shift;  activations have zero
//   point 0, so spatial padding is the integer 0;  4-bit tensors are packed two per byte along the
//   channel axis, even channel in bits 3:0, odd channel in bits 7:4, signed nibbles in two's
//   complement;  ReLU is applied after the residual add and before the clamp.
//
// Layouts: activations NHWC dense; weights [cout][kh][kw][cin]; all host pointers.
// Parity status of every exported function: pinned by tests/test_oracle_pins.py.

#include <cstdint>
#include <cstddef>
#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

enum { HQREF_OK = 0, HQREF_ERR_INVALID_ARG = 1, HQREF_ERR_RANGE = 4 };

// (x + 2^(c-1)) >> c with an arithmetic shift: round-half-up of x / 2^c.  1 <= c <= 62.
int64_t hqref_rshift_round(int64_t x, int32_t c) {
  const int64_t half = (int64_t)1 << (c - 1);
  return (x + half) >> c;
}

// Dyadic scaling of one integer: Int(q * b / 2^c)  (the DN(.) multiplier applied, Eq. 4).
int64_t hqref_dn(int32_t q, int32_t b, int32_t c) {
  return hqref_rshift_round((int64_t)q * (int64_t)b, c);
}

}  // extern "C"

namespace {

// Read element `idx` of a dense tensor stored with `bits` per element.
inline int64_t load_elem(const void* base, int64_t idx, int bits, int is_signed) {
  if (bits == 32) return (int64_t)((const int32_t*)base)[idx];
  if (bits == 8) {
    return is_signed ? (int64_t)((const int8_t*)base)[idx] : (int64_t)((const uint8_t*)base)[idx];
  }
  // bits == 4: two per byte, even element in the low nibble
  const uint8_t byte = ((const uint8_t*)base)[idx >> 1];
  int64_t v = (idx & 1) ? (int64_t)(byte >> 4) : (int64_t)(byte & 0x0F);
  if (is_signed && (v & 8)) v -= 16;
  return v;
}

// Write element `idx`; the value is already clamped to the representable range of the type.
inline void store_elem(void* base, int64_t idx, int bits, int is_signed, int64_t v) {
  if (bits == 32) { ((int32_t*)base)[idx] = (int32_t)v; return; }
  if (bits == 8) {
    if (is_signed) ((int8_t*)base)[idx] = (int8_t)v; else ((uint8_t*)base)[idx] = (uint8_t)v;
    return;
  }
  uint8_t* p = (uint8_t*)base + (idx >> 1);
  const uint8_t nib = (uint8_t)(v & 0x0F);
  if (idx & 1) *p = (uint8_t)((*p & 0x0F) | (nib << 4));
  else         *p = (uint8_t)((*p & 0xF0) | nib);
}

inline bool bits_ok(int bits, bool allow32) {
  return bits == 4 || bits == 8 || (allow32 && bits == 32);
}

inline bool dyadic_ok(const int32_t* b, const int32_t* c, int n) {
  if (!b || !c) return false;
  for (int i = 0; i < n; ++i) {
    if (b[i] < 0) return false;
    if (c[i] < 1 || c[i] > 62) return false;
  }
  return true;
}

inline bool fits_type(int64_t qmin, int64_t qmax, int bits, int is_signed) {
  int64_t lo, hi;
  if (bits == 32) { lo = -((int64_t)1 << 31); hi = ((int64_t)1 << 31) - 1; }
  else if (is_signed) { lo = -((int64_t)1 << (bits - 1)); hi = ((int64_t)1 << (bits - 1)) - 1; }
  else { lo = 0; hi = ((int64_t)1 << bits) - 1; }
  return qmin <= qmax && qmin >= lo && qmax <= hi;
}

}  // namespace

extern "C" {

// Quantized convolution layer, Eq. 3 + bias + Eq. 4 (+ residual, ReLU, clamp).
//
//   acc = sum_{r,s,ci} in[n, oh*stride + r - pad, ow*stride + s - pad, ci] * w[oc, r, s, ci]
//   t   = acc + bias[oc]                       (must fit INT32, else HQREF_ERR_RANGE)
//   out_bits == 32:  out = t
//   else             y = Int(t * b[oc] / 2^c[oc])
//                    if res:  y += Int(res * rb[oc] / 2^rc[oc])
//                    if relu: y = max(y, 0)
//                    out = clamp(y, qmin, qmax)
int32_t hqref_conv2d(const void* in, int32_t n, int32_t h, int32_t w, int32_t cin,
                     int32_t in_bits, int32_t in_signed,
                     const void* wgt, int32_t cout, int32_t kh, int32_t kw,
                     int32_t stride, int32_t pad, int32_t w_bits,
                     const int32_t* bias,
                     const int32_t* b, const int32_t* c,
                     const void* res, int32_t res_bits, int32_t res_signed,
                     const int32_t* rb, const int32_t* rc,
                     int32_t relu, int32_t qmin, int32_t qmax,
                     void* out, int32_t out_bits, int32_t out_signed) {
  if (!in || !wgt || !out) return HQREF_ERR_INVALID_ARG;
  if (n < 0 || h < 1 || w < 1 || cin < 1 || cout < 1 || kh < 1 || kw < 1 || stride < 1 || pad < 0)
    return HQREF_ERR_INVALID_ARG;
  if (!bits_ok(in_bits, false) || !bits_ok(w_bits, false) || !bits_ok(out_bits, true))
    return HQREF_ERR_INVALID_ARG;
  if (in_bits != w_bits) return HQREF_ERR_INVALID_ARG;       // b_w == b_a (Section 3.4, BOPS footnote)
  if (in_bits == 4 && (cin & 1)) return HQREF_ERR_INVALID_ARG;
  if (out_bits == 4 && (cout & 1)) return HQREF_ERR_INVALID_ARG;
  if (h + 2 * pad < kh || w + 2 * pad < kw) return HQREF_ERR_INVALID_ARG;
  if (out_bits != 32) {
    if (!dyadic_ok(b, c, cout)) return HQREF_ERR_INVALID_ARG;
    if (!fits_type(qmin, qmax, out_bits, out_signed)) return HQREF_ERR_INVALID_ARG;
    if (res) {
      if (!(res_bits == 8 || res_bits == 32)) return HQREF_ERR_INVALID_ARG;
      if (!dyadic_ok(rb, rc, cout)) return HQREF_ERR_INVALID_ARG;
    }
  }
  // output extent without a division: count the valid window positions
  int32_t oh_n = 0, ow_n = 0;
  for (int32_t y = 0; y + kh <= h + 2 * pad; y += stride) ++oh_n;
  for (int32_t x = 0; x + kw <= w + 2 * pad; x += stride) ++ow_n;

  int32_t status = HQREF_OK;
#pragma omp parallel for collapse(2) schedule(static)
  for (int32_t in_n = 0; in_n < n; ++in_n) {
    for (int32_t oh = 0; oh < oh_n; ++oh) {
      for (int32_t ow = 0; ow < ow_n; ++ow) {
        for (int32_t oc = 0; oc < cout; ++oc) {
          int64_t acc = 0;
          for (int32_t r = 0; r < kh; ++r) {
            const int32_t ih = oh * stride + r - pad;
            if (ih < 0 || ih >= h) continue;            // padded pixel contributes 0
            for (int32_t s = 0; s < kw; ++s) {
              const int32_t iw = ow * stride + s - pad;
              if (iw < 0 || iw >= w) continue;
              const int64_t in_base = (((int64_t)in_n * h + ih) * w + iw) * cin;
              const int64_t w_base = (((int64_t)oc * kh + r) * kw + s) * cin;
              for (int32_t ci = 0; ci < cin; ++ci) {
                acc += load_elem(in, in_base + ci, in_bits, in_signed) *
                       load_elem(wgt, w_base + ci, w_bits, 1);
              }
            }
          }
          const int64_t t = acc + (bias ? (int64_t)bias[oc] : 0);
          if (t < -((int64_t)1 << 31) || t > ((int64_t)1 << 31) - 1) {
#pragma omp atomic write
            status = HQREF_ERR_RANGE;
            continue;
          }
          const int64_t o_idx = (((int64_t)in_n * oh_n + oh) * ow_n + ow) * cout + oc;
          if (out_bits == 32) {
            store_elem(out, o_idx, 32, 1, t);
            continue;
          }
          int64_t y = hqref_dn((int32_t)t, b[oc], c[oc]);
          if (res) {
            const int64_t q_r = load_elem(res, o_idx, res_bits, res_signed);
            y += hqref_dn((int32_t)q_r, rb[oc], rc[oc]);
          }
          if (relu && y < 0) y = 0;
          if (y < qmin) y = qmin;
          if (y > qmax) y = qmax;
          store_elem(out, o_idx, out_bits, out_signed, y);
        }
      }
    }
  }
  return status;
}

// Fully connected layer: a convolution whose spatial extent is 1x1 (Eq. 3 as a matrix product).
int32_t hqref_linear(const void* in, int32_t n, int32_t cin, int32_t in_bits, int32_t in_signed,
                     const void* wgt, int32_t cout, int32_t w_bits, const int32_t* bias,
                     const int32_t* b, const int32_t* c,
                     int32_t relu, int32_t qmin, int32_t qmax,
                     void* out, int32_t out_bits, int32_t out_signed) {
  return hqref_conv2d(in, n, 1, 1, cin, in_bits, in_signed, wgt, cout, 1, 1, 1, 0, w_bits, bias,
                      b, c, nullptr, 0, 0, nullptr, nullptr, relu, qmin, qmax,
                      out, out_bits, out_signed);
}

// Residual add on stored tensors (Section 3.3):
//   y = Int(main * mb[ch] / 2^mc[ch]) + (res ? Int(res * rb[ch] / 2^rc[ch]) : 0); ReLU; clamp.
// With res == NULL this is a plain dyadic requantization of `main`.
int32_t hqref_residual_add(const void* main_t, int32_t main_bits, int32_t main_signed,
                           const int32_t* mb, const int32_t* mc,
                           const void* res, int32_t res_bits, int32_t res_signed,
                           const int32_t* rb, const int32_t* rc,
                           int64_t pixels, int32_t ch,
                           int32_t relu, int32_t qmin, int32_t qmax,
                           void* out, int32_t out_bits, int32_t out_signed) {
  if (!main_t || !out || pixels < 0 || ch < 1) return HQREF_ERR_INVALID_ARG;
  // out_bits == 32: the sum stays a wide integer (the INT32 residual stream of Fig. 2), clamped to [qmin, qmax]
  if (!bits_ok(main_bits, true) || !bits_ok(out_bits, true)) return HQREF_ERR_INVALID_ARG;
  if ((main_bits == 4 || out_bits == 4) && (ch & 1)) return HQREF_ERR_INVALID_ARG;
  if (!dyadic_ok(mb, mc, ch)) return HQREF_ERR_INVALID_ARG;
  if (res && (!bits_ok(res_bits, true) || !dyadic_ok(rb, rc, ch))) return HQREF_ERR_INVALID_ARG;
  if (res && res_bits == 4 && (ch & 1)) return HQREF_ERR_INVALID_ARG;
  if (!fits_type(qmin, qmax, out_bits, out_signed)) return HQREF_ERR_INVALID_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < pixels; ++p) {
    for (int32_t k = 0; k < ch; ++k) {
      const int64_t idx = p * ch + k;
      int64_t y = hqref_dn((int32_t)load_elem(main_t, idx, main_bits, main_signed), mb[k], mc[k]);
      if (res) y += hqref_dn((int32_t)load_elem(res, idx, res_bits, res_signed), rb[k], rc[k]);
      if (relu && y < 0) y = 0;
      if (y < qmin) y = qmin;
      if (y > qmax) y = qmax;
      store_elem(out, idx, out_bits, out_signed, y);
    }
  }
  return HQREF_OK;
}

// Global average pooling on wide integers (Appendix E), with no division: the sum over the h*w
// pixels is kept wide and the factor 1/(h*w) is part of the dyadic multiplier b / 2^c.
int32_t hqref_avgpool_requant(const void* in, int32_t n, int32_t h, int32_t w, int32_t ch,
                              int32_t in_bits, int32_t in_signed,
                              const int32_t* b, const int32_t* c,
                              int32_t qmin, int32_t qmax,
                              void* out, int32_t out_bits, int32_t out_signed) {
  if (!in || !out || n < 0 || h < 1 || w < 1 || ch < 1) return HQREF_ERR_INVALID_ARG;
  if (!bits_ok(in_bits, true) || !bits_ok(out_bits, false)) return HQREF_ERR_INVALID_ARG;
  if ((in_bits == 4 || out_bits == 4) && (ch & 1)) return HQREF_ERR_INVALID_ARG;
  if (!dyadic_ok(b, c, ch)) return HQREF_ERR_INVALID_ARG;
  if (!fits_type(qmin, qmax, out_bits, out_signed)) return HQREF_ERR_INVALID_ARG;
  int32_t status = HQREF_OK;
  for (int32_t in_n = 0; in_n < n; ++in_n) {
    for (int32_t k = 0; k < ch; ++k) {
      int64_t sum = 0;
      for (int32_t y = 0; y < h; ++y)
        for (int32_t x = 0; x < w; ++x)
          sum += load_elem(in, (((int64_t)in_n * h + y) * w + x) * ch + k, in_bits, in_signed);
      if (sum < -((int64_t)1 << 31) || sum > ((int64_t)1 << 31) - 1) { status = HQREF_ERR_RANGE; continue; }
      int64_t q = hqref_dn((int32_t)sum, b[k], c[k]);
      if (q < qmin) q = qmin;
      if (q > qmax) q = qmax;
      store_elem(out, (int64_t)in_n * ch + k, out_bits, out_signed, q);
    }
  }
  return status;
}

// Max pooling over a k x k window on a stored 8-bit tensor; taps outside the image are skipped.
int32_t hqref_maxpool(const void* in, int32_t n, int32_t h, int32_t w, int32_t ch,
                      int32_t bits, int32_t is_signed,
                      int32_t k, int32_t stride, int32_t pad, void* out) {
  if (!in || !out || n < 0 || h < 1 || w < 1 || ch < 1 || k < 1 || stride < 1 || pad < 0)
    return HQREF_ERR_INVALID_ARG;
  if (bits != 8 && bits != 32) return HQREF_ERR_INVALID_ARG;   // 32: pooling on the wide feature map (Appendix E)
  if (pad >= k) return HQREF_ERR_INVALID_ARG;   // every window must touch the image
  int32_t oh_n = 0, ow_n = 0;
  for (int32_t y = 0; y + k <= h + 2 * pad; y += stride) ++oh_n;
  for (int32_t x = 0; x + k <= w + 2 * pad; x += stride) ++ow_n;
#pragma omp parallel for collapse(2) schedule(static)
  for (int32_t in_n = 0; in_n < n; ++in_n) {
    for (int32_t oh = 0; oh < oh_n; ++oh) {
      for (int32_t ow = 0; ow < ow_n; ++ow) {
        for (int32_t cc = 0; cc < ch; ++cc) {
          bool any = false;
          int64_t best = 0;
          for (int32_t r = 0; r < k; ++r) {
            const int32_t ih = oh * stride + r - pad;
            if (ih < 0 || ih >= h) continue;
            for (int32_t s = 0; s < k; ++s) {
              const int32_t iw = ow * stride + s - pad;
              if (iw < 0 || iw >= w) continue;
              const int64_t v = load_elem(in, (((int64_t)in_n * h + ih) * w + iw) * ch + cc, bits, is_signed);
              if (!any || v > best) { best = v; any = true; }
            }
          }
          store_elem(out, (((int64_t)in_n * oh_n + oh) * ow_n + ow) * ch + cc, bits, is_signed, best);
        }
      }
    }
  }
  return HQREF_OK;
}

// One branch of an Inception-style concatenation (Appendix E, "Concatenation Layer"): every branch
// is brought to the output scale by its own dyadic pairs, q_a[.., off + k] = DN(S_i / S_a) q_i[.., k],
// and lands beside the others along the channel axis; the convolution branches arrive as stored
// 8-bit (or 4-bit) tensors or as wide accumulators, the pooling branch as a wide (INT32) tensor.
// `out` is the [pixels][out_ch] concatenated tensor, `ch_off` the branch's first channel in it.
int32_t hqref_concat_branch(const void* in, int32_t in_bits, int32_t in_signed,
                            const int32_t* b, const int32_t* c, int64_t pixels, int32_t ch,
                            int32_t relu, int32_t qmin, int32_t qmax,
                            void* out, int32_t out_bits, int32_t out_signed, int32_t out_ch, int32_t ch_off) {
  if (!in || !out || pixels < 0 || ch < 1 || ch_off < 0 || out_ch < ch_off + ch) return HQREF_ERR_INVALID_ARG;
  if (!bits_ok(in_bits, true) || !bits_ok(out_bits, false)) return HQREF_ERR_INVALID_ARG;
  if (in_bits == 4 && (ch & 1)) return HQREF_ERR_INVALID_ARG;
  if (out_bits == 4 && (out_ch & 1)) return HQREF_ERR_INVALID_ARG;
  if (!dyadic_ok(b, c, ch)) return HQREF_ERR_INVALID_ARG;
  if (!fits_type(qmin, qmax, out_bits, out_signed)) return HQREF_ERR_INVALID_ARG;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < pixels; ++p) {
    for (int32_t k = 0; k < ch; ++k) {
      int64_t y = hqref_dn((int32_t)load_elem(in, p * ch + k, in_bits, in_signed), b[k], c[k]);
      if (relu && y < 0) y = 0;
      if (y < qmin) y = qmin;
      if (y > qmax) y = qmax;
      store_elem(out, p * out_ch + ch_off + k, out_bits, out_signed, y);
    }
  }
  return HQREF_OK;
}

// Windowed sum pooling on wide integers (Appendix E: the pooling branch of an Inception module stays in
// INT32): out[n,oh,ow,c] = sum over the k x k window of in[n, oh*stride+r-pad, ow*stride+s-pad, c], taps
// outside the image counting as 0; the reciprocal of the window size of an average pool belongs to the dyadic pair of the
// consumer (no division, Section 1).  in: bits 4/8/32; out: INT32 [n, oh, ow, c].
int32_t hqref_sumpool(const void* in, int32_t n, int32_t h, int32_t w, int32_t ch, int32_t bits, int32_t is_signed,
                      int32_t k, int32_t stride, int32_t pad, int32_t* out) {
  if (!in || !out || n < 0 || h < 1 || w < 1 || ch < 1 || k < 1 || stride < 1 || pad < 0 || pad >= k)
    return HQREF_ERR_INVALID_ARG;
  if (!bits_ok(bits, true) || (bits == 4 && (ch & 1))) return HQREF_ERR_INVALID_ARG;
  if (h + 2 * pad < k || w + 2 * pad < k) return HQREF_ERR_INVALID_ARG;
  int32_t oh_n = 0, ow_n = 0;                      // window positions, counted (no division anywhere in this file)
  for (int32_t y = 0; y + k <= h + 2 * pad; y += stride) ++oh_n;
  for (int32_t x = 0; x + k <= w + 2 * pad; x += stride) ++ow_n;
  int32_t status = HQREF_OK;
#pragma omp parallel for schedule(static)
  for (int32_t in_n = 0; in_n < n; ++in_n) {
    for (int32_t oh = 0; oh < oh_n; ++oh) {
      for (int32_t ow = 0; ow < ow_n; ++ow) {
        for (int32_t cc = 0; cc < ch; ++cc) {
          int64_t sum = 0;
          for (int32_t r = 0; r < k; ++r) {
            const int32_t ih = oh * stride + r - pad;
            if (ih < 0 || ih >= h) continue;
            for (int32_t s = 0; s < k; ++s) {
              const int32_t iw = ow * stride + s - pad;
              if (iw < 0 || iw >= w) continue;
              sum += load_elem(in, (((int64_t)in_n * h + ih) * w + iw) * ch + cc, bits, is_signed);
            }
          }
          if (sum < INT32_MIN || sum > INT32_MAX) {
#pragma omp atomic write
            status = HQREF_ERR_RANGE;
            sum = 0;
          }
          out[(((int64_t)in_n * oh_n + oh) * ow_n + ow) * ch + cc] = (int32_t)sum;
        }
      }
    }
  }
  return status;
}

int32_t hqref_num_threads(void) {
  int32_t t = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp master
    t = omp_get_num_threads();
  }
#endif
  return t;
}

}  // extern "C"
