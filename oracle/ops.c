/*
 * CPU oracle: plain definitions of the operators on the fused-CNN hot path.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing in the product (the CUDA library and its Python
 * binding) may include, link or call this file; it shares no code with the CUDA path.
 * It is meant to be checked against the paper by eye: every routine is the textbook
 * definition written as nested loops, with no blocking, fusion or reordering.
 *
 * Conventions: logical tensors are NHWC float (fp32 storage); every accumulation is
 * carried in double and rounded to float once.  The paper defines convolution only
 * verbally (Section 4, "For a 2D Convolution": each output element iterates over the
 * kernel window and the input channels under it), so these are the standard
 * definitions of that sentence.
 *
 * OpenMP splits the outermost (batch x output row) loop only; each output element is
 * still produced by one thread with the loop order given here.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
int orc_num_threads(void) { return omp_get_max_threads(); }
void orc_set_threads(int n) { omp_set_num_threads(n); }
#else
int orc_num_threads(void) { return 1; }
void orc_set_threads(int n) { (void)n; }
#endif

/* Output extent of a strided, dilated, padded window (standard formula). */
int orc_out_size(int in, int k, int stride, int dilation, int pad_before, int pad_after) {
  return (in + pad_before + pad_after - ((k - 1) * dilation + 1)) / stride + 1;
}

/*
 * Full convolution (Section 4, "For a 2D Convolution").
 *   out[b,oy,ox,co] = bias[co] + sum_{ky,kx,ci} x[b, oy*sh - pt + ky*dh, ox*sw - pl + kx*dw, ci] * w[co,ky,kx,ci]
 * Out-of-range x reads as zero.  w is [Cout][kh][kw][Cin]; bias may be NULL.
 */
void orc_conv2d(const float* x, int B, int H, int W, int Cin, const float* w, const float* bias, int Cout, int kh,
                int kw, int sh, int sw, int dh, int dw, int pt, int pl, int pb, int pr, float* out) {
  const int Ho = orc_out_size(H, kh, sh, dh, pt, pb);
  const int Wo = orc_out_size(W, kw, sw, dw, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int oy = 0; oy < Ho; ++oy)
      for (int ox = 0; ox < Wo; ++ox)
        for (int co = 0; co < Cout; ++co) {
          double acc = bias ? (double)bias[co] : 0.0;
          for (int ky = 0; ky < kh; ++ky) {
            const int iy = oy * sh - pt + ky * dh;
            if (iy < 0 || iy >= H) continue;
            for (int kx = 0; kx < kw; ++kx) {
              const int ix = ox * sw - pl + kx * dw;
              if (ix < 0 || ix >= W) continue;
              const float* xp = x + (((size_t)b * H + iy) * W + ix) * Cin;
              const float* wp = w + (((size_t)co * kh + ky) * kw + kx) * Cin;
              for (int ci = 0; ci < Cin; ++ci) acc += (double)xp[ci] * (double)wp[ci];
            }
          }
          out[(((size_t)b * Ho + oy) * Wo + ox) * Cout + co] = (float)acc;
        }
}

/*
 * Depthwise convolution, depth multiplier 1: the same sum with co = ci = c and one
 * filter per channel.  w is [kh][kw][C].
 */
void orc_depthwise(const float* x, int B, int H, int W, int C, const float* w, const float* bias, int kh, int kw,
                   int sh, int sw, int dh, int dw, int pt, int pl, int pb, int pr, float* out) {
  const int Ho = orc_out_size(H, kh, sh, dh, pt, pb);
  const int Wo = orc_out_size(W, kw, sw, dw, pl, pr);
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int oy = 0; oy < Ho; ++oy)
      for (int ox = 0; ox < Wo; ++ox)
        for (int c = 0; c < C; ++c) {
          double acc = bias ? (double)bias[c] : 0.0;
          for (int ky = 0; ky < kh; ++ky) {
            const int iy = oy * sh - pt + ky * dh;
            if (iy < 0 || iy >= H) continue;
            for (int kx = 0; kx < kw; ++kx) {
              const int ix = ox * sw - pl + kx * dw;
              if (ix < 0 || ix >= W) continue;
              acc += (double)x[(((size_t)b * H + iy) * W + ix) * C + c] * (double)w[((size_t)ky * kw + kx) * C + c];
            }
          }
          out[(((size_t)b * Ho + oy) * Wo + ox) * C + c] = (float)acc;
        }
}

/* Element-wise successors (Section 3.2: activations are what gets fused into convolutions). */
void orc_relu(float* x, size_t n) {
  for (size_t i = 0; i < n; ++i) x[i] = x[i] > 0.0f ? x[i] : 0.0f;
}
void orc_relu6(float* x, size_t n) {
  for (size_t i = 0; i < n; ++i) {
    float v = x[i] > 0.0f ? x[i] : 0.0f;
    x[i] = v < 6.0f ? v : 6.0f;
  }
}
void orc_add(const float* a, const float* b, float* out, size_t n) {
  for (size_t i = 0; i < n; ++i) out[i] = a[i] + b[i];
}

/* Mean over H*W per (image, channel). */
void orc_global_avg_pool(const float* x, int B, int H, int W, int C, float* out) {
  for (int b = 0; b < B; ++b)
    for (int c = 0; c < C; ++c) {
      double acc = 0.0;
      for (int p = 0; p < H * W; ++p) acc += (double)x[((size_t)b * H * W + p) * C + c];
      out[(size_t)b * C + c] = (float)(acc / (double)(H * W));
    }
}

/*
 * Bilinear resize.  align_corners: src = o * (in-1)/(out-1); otherwise src = o * in/out.
 * i0 = floor(src), i1 = min(i0+1, in-1), weight = src - i0; interpolate along x, then y.
 */
void orc_resize_bilinear(const float* x, int B, int H, int W, int C, float* out, int OH, int OW, int align_corners) {
  const double sy = align_corners ? (OH > 1 ? (double)(H - 1) / (double)(OH - 1) : 0.0) : (double)H / (double)OH;
  const double sx = align_corners ? (OW > 1 ? (double)(W - 1) / (double)(OW - 1) : 0.0) : (double)W / (double)OW;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int oy = 0; oy < OH; ++oy) {
      const double fy = oy * sy;
      int y0 = (int)floor(fy);
      if (y0 > H - 1) y0 = H - 1;
      const int y1 = y0 + 1 < H ? y0 + 1 : H - 1;
      const double wy = fy - y0;
      for (int ox = 0; ox < OW; ++ox) {
        const double fx = ox * sx;
        int x0 = (int)floor(fx);
        if (x0 > W - 1) x0 = W - 1;
        const int x1 = x0 + 1 < W ? x0 + 1 : W - 1;
        const double wx = fx - x0;
        for (int c = 0; c < C; ++c) {
          const double v00 = x[(((size_t)b * H + y0) * W + x0) * C + c];
          const double v01 = x[(((size_t)b * H + y0) * W + x1) * C + c];
          const double v10 = x[(((size_t)b * H + y1) * W + x0) * C + c];
          const double v11 = x[(((size_t)b * H + y1) * W + x1) * C + c];
          const double top = v00 + (v01 - v00) * wx;
          const double bot = v10 + (v11 - v10) * wx;
          out[(((size_t)b * OH + oy) * OW + ox) * C + c] = (float)(top + (bot - top) * wy);
        }
      }
    }
}

/*
 * fp32 -> fp16 bits, IEEE round-to-nearest-even, subnormals kept, overflow to infinity.
 * Written on the bit patterns so it does not depend on compiler half support.
 */
uint16_t orc_f32_to_f16_bits_1(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  const uint32_t sign = (u >> 16) & 0x8000u;
  const uint32_t absu = u & 0x7fffffffu;
  if (absu >= 0x7f800000u) /* inf or nan */
    return (uint16_t)(sign | 0x7c00u | (absu > 0x7f800000u ? 0x0200u | ((absu >> 13) & 0x3ffu) : 0u));
  const int32_t e = (int32_t)(absu >> 23) - 127; /* unbiased exponent */
  uint32_t man = absu & 0x7fffffu;
  if (e > 15) return (uint16_t)(sign | 0x7c00u); /* too large even before rounding */
  if (e >= -14) {
    /* normal half: keep 10 mantissa bits, round on the 13 dropped ones */
    uint32_t h = ((uint32_t)(e + 15) << 10) | (man >> 13);
    const uint32_t rem = man & 0x1fffu;
    if (rem > 0x1000u || (rem == 0x1000u && (h & 1u))) ++h; /* may carry into exponent, up to inf: correct */
    return (uint16_t)(sign | h);
  }
  if (e < -25) return (uint16_t)sign; /* below half of the smallest subnormal: rounds to zero */
  /* subnormal half: value = man_full * 2^(e-23); unit is 2^-24 */
  man |= 0x800000u;
  const int shift = -e - 1; /* 14..24: man_full >> shift is the count of 2^-24 units */
  uint32_t h = man >> shift;
  const uint32_t rem = man & ((1u << shift) - 1u);
  const uint32_t half = 1u << (shift - 1);
  if (rem > half || (rem == half && (h & 1u))) ++h;
  return (uint16_t)(sign | h);
}

float orc_f16_bits_to_f32_1(uint16_t h) {
  const uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  const uint32_t e = (h >> 10) & 0x1fu;
  const uint32_t m = h & 0x3ffu;
  float r;
  if (e == 0) {
    r = ldexpf((float)m, -24);
  } else if (e == 31) {
    uint32_t u = 0x7f800000u | (m << 13);
    memcpy(&r, &u, 4);
  } else {
    r = ldexpf((float)(m | 0x400u), (int)e - 25);
  }
  uint32_t u;
  memcpy(&u, &r, 4);
  u |= sign;
  memcpy(&r, &u, 4);
  return r;
}

void orc_f32_to_f16_bits(const float* x, uint16_t* out, size_t n) {
  for (size_t i = 0; i < n; ++i) out[i] = orc_f32_to_f16_bits_1(x[i]);
}
void orc_f16_bits_to_f32(const uint16_t* x, float* out, size_t n) {
  for (size_t i = 0; i < n; ++i) out[i] = orc_f16_bits_to_f32_1(x[i]);
}
/* Storage emulation: the value a tensor holds after being written as fp16 and read back. */
void orc_round_f16(float* x, size_t n) {
  for (size_t i = 0; i < n; ++i) x[i] = orc_f16_bits_to_f32_1(orc_f32_to_f16_bits_1(x[i]));
}

/*
 * PHWC4 (Section 4, "Data Layout", and Fig. 1): a [H,W,C] tensor is cut into ceil(C/4)
 * slices of shape (H, W, 4) stored one after another; missing channels are zero.
 * Batches: the paper treats a batch as a concatenation of [H,W,C] tensors; here the B
 * planes of one slice are concatenated, then the slices ([S][B][plane][4]).  A plane
 * holds plane_pixels >= H*W pixels (the caller passes H*W rounded up to even, so a
 * plane is a whole number of 16-byte fp16 units); the extra pixel is zero.
 */
size_t orc_phwc4_index(int B, int H, int W, int plane_pixels, int b, int h, int w, int c) {
  (void)H;
  const int s = c / 4;
  return (((size_t)s * B + b) * plane_pixels + (size_t)h * W + w) * 4 + (size_t)(c % 4);
}
void orc_phwc4_pack(const float* nhwc, int B, int H, int W, int C, int plane_pixels, float* out) {
  const int S = (C + 3) / 4;
  memset(out, 0, (size_t)S * B * plane_pixels * 4 * sizeof(float));
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h)
      for (int w = 0; w < W; ++w)
        for (int c = 0; c < C; ++c)
          out[orc_phwc4_index(B, H, W, plane_pixels, b, h, w, c)] = nhwc[(((size_t)b * H + h) * W + w) * C + c];
}
void orc_phwc4_unpack(const float* phwc4, int B, int H, int W, int C, int plane_pixels, float* nhwc) {
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h)
      for (int w = 0; w < W; ++w)
        for (int c = 0; c < C; ++c)
          nhwc[(((size_t)b * H + h) * W + w) * C + c] = phwc4[orc_phwc4_index(B, H, W, plane_pixels, b, h, w, c)];
}
