/*
 * CPU oracle for the tool-tracking per-frame hot path.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is a plain, slow, definition-level implementation of every stage of the
 * pipeline the paper's Endoscopy Tool Tracking application runs per frame
 * (Section III-A: format conversion -> recurrent inference -> tool-tracking
 * post-processing -> overlay).  The paper fixes the operator chain but none of the
 * arithmetic; the arithmetic below is the textbook definition of each stage, written out
 * as nested loops with double-precision accumulation and one rounding to fp32 per stored
 * value.  There is no blocking, fusion, vectorisation or reordering; the optional OpenMP
 * pragmas only distribute independent output elements over host threads.
 *
 * Nothing here is shared with, derived from, or used by the CUDA implementation.  Only
 * tests, the smoke check and the benchmark's CPU-baseline leg may call into it.
 *
 * Parity pins (tests/test_oracle_*.py): resize fixed points and a rational brute force,
 * direct convolution re-derived in scatter form plus delta/ones kernels, ConvLSTM closed
 * forms (zero weights, saturated gates), sigmoid identities, hand-computed centroids and
 * blends.  The composed pipeline has no externally published value to compare with (the
 * paper prints no tensor): whole-pipeline parity is pinned stage by stage only.
 */
#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int ora_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void ora_set_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

/* ------------------------------------------------------------------------------------
 * O1  bilinear resize with half-pixel centres, edge clamp, no antialiasing.
 *
 * Output sample o of an axis resized from `in` to `out` samples sits at source position
 * s = (o + 1/2) * in/out - 1/2.  Written as an exact rational: s = num/den with
 * num = (2o+1)*in - out and den = 2*out, clamped to [0, in-1].  i0 = floor(s), i1 = min(i0+1,
 * in-1), frac = s - i0.  All of this is integer arithmetic, hence reproducible bit for bit.
 * ------------------------------------------------------------------------------------ */
void ora_resize_axis(int in, int out, int32_t* i0, int32_t* i1, double* frac) {
  for (int o = 0; o < out; ++o) {
    int64_t den = 2 * (int64_t)out;
    int64_t num = (2 * (int64_t)o + 1) * (int64_t)in - (int64_t)out;
    int64_t hi = ((int64_t)in - 1) * den;
    if (num < 0) num = 0;
    if (num > hi) num = hi;
    int64_t lo_idx = num / den;
    int64_t up_idx = lo_idx + 1 < in ? lo_idx + 1 : in - 1;
    i0[o] = (int32_t)lo_idx;
    i1[o] = (int32_t)up_idx;
    frac[o] = (double)(num - lo_idx * den) / (double)den;
  }
}

/* uint8 HWC RGB (row pitch in bytes) -> resized, normalised fp32 planar [3][net_h][net_w].
 * value = ((v/div) - mean)/std with v the bilinear sample on the raw 0..255 scale. */
void ora_preprocess(const uint8_t* src, int src_w, int src_h, int src_pitch, int net_w, int net_h,
                    double norm_div, double norm_mean, double norm_std, float* dst,
                    int32_t* x0, int32_t* x1, double* fx, int32_t* y0, int32_t* y1, double* fy) {
  ora_resize_axis(src_w, net_w, x0, x1, fx);
  ora_resize_axis(src_h, net_h, y0, y1, fy);
  for (int c = 0; c < 3; ++c)
    for (int yo = 0; yo < net_h; ++yo)
      for (int xo = 0; xo < net_w; ++xo) {
        const uint8_t* r0 = src + (size_t)y0[yo] * src_pitch;
        const uint8_t* r1 = src + (size_t)y1[yo] * src_pitch;
        double p00 = r0[3 * x0[xo] + c], p01 = r0[3 * x1[xo] + c];
        double p10 = r1[3 * x0[xo] + c], p11 = r1[3 * x1[xo] + c];
        double top = p00 + fx[xo] * (p01 - p00);
        double bot = p10 + fx[xo] * (p11 - p10);
        double v = top + fy[yo] * (bot - top);
        dst[((size_t)c * net_h + yo) * net_w + xo] = (float)(((v / norm_div) - norm_mean) / norm_std);
      }
}

/* ------------------------------------------------------------------------------------
 * O2  3x3 cross-correlation, zero padding 1 on every side, stride s, bias, optional ReLU.
 *   y[o][yo][xo] = b[o] + sum_c sum_ky sum_kx w[o][c][ky][kx] * in[c][yo*s+ky-1][xo*s+kx-1]
 * Output extent floor((n + 2 - 3)/s) + 1.  Planar (NCHW without N) fp32 in and out, OIHW
 * weights, double accumulator, one rounding to fp32.
 * ------------------------------------------------------------------------------------ */
int ora_conv_out(int n, int stride) { return (n + 2 - 3) / stride + 1; }

void ora_conv3x3(const float* in, int cin, int h, int w, const float* wgt, const float* bias,
                 int cout, int stride, int relu, float* out) {
  int ho = ora_conv_out(h, stride), wo = ora_conv_out(w, stride);
#pragma omp parallel for collapse(2) schedule(static)
  for (int o = 0; o < cout; ++o)
    for (int yo = 0; yo < ho; ++yo)
      for (int xo = 0; xo < wo; ++xo) {
        double acc = bias ? (double)bias[o] : 0.0;
        for (int c = 0; c < cin; ++c)
          for (int ky = 0; ky < 3; ++ky)
            for (int kx = 0; kx < 3; ++kx) {
              int yi = yo * stride + ky - 1, xi = xo * stride + kx - 1;
              if (yi < 0 || yi >= h || xi < 0 || xi >= w) continue;
              acc += (double)wgt[(((size_t)o * cin + c) * 3 + ky) * 3 + kx] *
                     (double)in[((size_t)c * h + yi) * w + xi];
            }
        if (relu && acc < 0.0) acc = 0.0;
        out[((size_t)o * ho + yo) * wo + xo] = (float)acc;
      }
}

/* ------------------------------------------------------------------------------------
 * O3  ConvLSTM cell step (Shi et al. 2015 form without peepholes).
 *   [i|f|g|o] = W (*) concat[x, h] + b   (3x3, stride 1, pad 1; 4*ch output maps in blocks)
 *   c' = sigmoid(f)*c + sigmoid(i)*tanh(g);   h' = sigmoid(o)*tanh(c')
 * x: [cx][hm][wm], h,c: [ch][hm][wm]; W: [4ch][cx+ch][3][3] with input channels x first.
 * `gates` (optional, may be NULL) receives the 4*ch pre-activation maps as fp32.
 * ------------------------------------------------------------------------------------ */
static double sigmoid_d(double z) { return 1.0 / (1.0 + exp(-z)); }

void ora_convlstm_step(const float* x, int cx, const float* h, const float* c, int ch, int hm,
                       int wm, const float* wgt, const float* bias, float* h_out, float* c_out,
                       float* gates) {
  int cin = cx + ch;
  size_t plane = (size_t)hm * wm;
#pragma omp parallel for collapse(2) schedule(static)
  for (int j = 0; j < ch; ++j)
    for (int yo = 0; yo < hm; ++yo)
      for (int xo = 0; xo < wm; ++xo) {
        double pre[4];
        for (int g = 0; g < 4; ++g) {
          int o = g * ch + j;
          double acc = bias ? (double)bias[o] : 0.0;
          for (int ci = 0; ci < cin; ++ci) {
            const float* src = ci < cx ? x + (size_t)ci * plane : h + (size_t)(ci - cx) * plane;
            for (int ky = 0; ky < 3; ++ky)
              for (int kx = 0; kx < 3; ++kx) {
                int yi = yo + ky - 1, xi = xo + kx - 1;
                if (yi < 0 || yi >= hm || xi < 0 || xi >= wm) continue;
                acc += (double)wgt[(((size_t)o * cin + ci) * 3 + ky) * 3 + kx] *
                       (double)src[(size_t)yi * wm + xi];
              }
          }
          pre[g] = acc;
          if (gates) gates[(size_t)o * plane + (size_t)yo * wm + xo] = (float)acc;
        }
        size_t idx = (size_t)j * plane + (size_t)yo * wm + xo;
        double cn = sigmoid_d(pre[1]) * (double)c[idx] + sigmoid_d(pre[0]) * tanh(pre[2]);
        float cn_f = (float)cn;                 /* the state is stored in fp32 */
        c_out[idx] = cn_f;
        h_out[idx] = (float)(sigmoid_d(pre[3]) * tanh((double)cn_f));
      }
}

/* ------------------------------------------------------------------------------------
 * O4  mask head: z_t = b_t + sum_j w[t][j]*h[j];  p = sigmoid(z);  mask = z > logit(thr)
 * (strict).  The comparison is taken on the fp32 logit.
 * ------------------------------------------------------------------------------------ */
void ora_head(const float* h, int ch, int hm, int wm, const float* wgt, const float* bias, int T,
              double thr, float* z, float* p, uint8_t* mask) {
  size_t plane = (size_t)hm * wm;
  float zthr = (float)log(thr / (1.0 - thr));
  for (int t = 0; t < T; ++t)
    for (size_t i = 0; i < plane; ++i) {
      double acc = bias ? (double)bias[t] : 0.0;
      for (int j = 0; j < ch; ++j) acc += (double)wgt[(size_t)t * ch + j] * (double)h[(size_t)j * plane + i];
      float zf = (float)acc;
      z[(size_t)t * plane + i] = zf;
      p[(size_t)t * plane + i] = (float)sigmoid_d((double)zf);
      mask[(size_t)t * plane + i] = zf > zthr ? 1 : 0;
    }
}

/* ------------------------------------------------------------------------------------
 * O5  per-tool confidence and mask centroid.
 *   mean-sigmoid:  conf_t = mean over the grid of p_t
 *   gap-linear:    conf_t = sigmoid(b_t + sum_j w[t][j] * mean_grid(h[j]))
 *   centroid:      (sum x, sum y)/count over mask_t == 1 in grid index coordinates;
 *                  an empty mask gives (-1, -1) and count 0.
 * ------------------------------------------------------------------------------------ */
void ora_conf_mean_sigmoid(const float* p, int T, int hm, int wm, float* conf) {
  size_t plane = (size_t)hm * wm;
  for (int t = 0; t < T; ++t) {
    double s = 0.0;
    for (size_t i = 0; i < plane; ++i) s += (double)p[(size_t)t * plane + i];
    conf[t] = (float)(s / (double)plane);
  }
}

void ora_conf_gap_linear(const float* h, int ch, int hm, int wm, const float* wgt, const float* bias,
                         int T, float* conf) {
  size_t plane = (size_t)hm * wm;
  for (int t = 0; t < T; ++t) {
    double acc = bias ? (double)bias[t] : 0.0;
    for (int j = 0; j < ch; ++j) {
      double s = 0.0;
      for (size_t i = 0; i < plane; ++i) s += (double)h[(size_t)j * plane + i];
      acc += (double)wgt[(size_t)t * ch + j] * (s / (double)plane);
    }
    conf[t] = (float)sigmoid_d(acc);
  }
}

void ora_centroids(const uint8_t* mask, int T, int hm, int wm, float* cx, float* cy, int32_t* count) {
  for (int t = 0; t < T; ++t) {
    int64_t n = 0, sx = 0, sy = 0;
    for (int y = 0; y < hm; ++y)
      for (int x = 0; x < wm; ++x)
        if (mask[((size_t)t * hm + y) * wm + x]) { n += 1; sx += x; sy += y; }
    count[t] = (int32_t)n;
    cx[t] = n ? (float)((double)sx / (double)n) : -1.0f;
    cy[t] = n ? (float)((double)sy / (double)n) : -1.0f;
  }
}

/* ------------------------------------------------------------------------------------
 * O6  overlay (stands in for the visualisation load): RGBA8 copy of the source frame;
 * mask grid nearest-upsampled by integer floor; tools blended in ascending order with
 * alpha = 102/255 = 0.4 in rounded integer arithmetic; output alpha 255.
 * ------------------------------------------------------------------------------------ */
void ora_overlay(const uint8_t* src, int src_w, int src_h, int src_pitch, const uint8_t* mask, int T,
                 int hm, int wm, const uint8_t* palette /*[T][3]*/, uint8_t* dst /*[src_h][src_w][4]*/) {
  for (int y = 0; y < src_h; ++y)
    for (int x = 0; x < src_w; ++x) {
      int mx = (int)(((int64_t)x * wm) / src_w), my = (int)(((int64_t)y * hm) / src_h);
      int rgb[3];
      for (int k = 0; k < 3; ++k) rgb[k] = src[(size_t)y * src_pitch + 3 * x + k];
      for (int t = 0; t < T; ++t)
        if (mask[((size_t)t * hm + my) * wm + mx])
          for (int k = 0; k < 3; ++k) rgb[k] = (153 * rgb[k] + 102 * (int)palette[3 * t + k] + 127) / 255;
      uint8_t* o = dst + ((size_t)y * src_w + x) * 4;
      o[0] = (uint8_t)rgb[0]; o[1] = (uint8_t)rgb[1]; o[2] = (uint8_t)rgb[2]; o[3] = 255;
    }
}

/* Round-to-nearest-even fp32 -> bf16 -> fp32 on an array, used only by the variant of the
 * pipeline that mirrors where a bf16 tensor-core path rounds its activations. */
void ora_round_bf16(float* a, size_t n) {
  for (size_t i = 0; i < n; ++i) {
    uint32_t u; memcpy(&u, &a[i], 4);
    if ((u & 0x7F800000u) != 0x7F800000u) {
      u += 0x7FFFu + ((u >> 16) & 1u);
      u &= 0xFFFF0000u;
    }
    memcpy(&a[i], &u, 4);
  }
}
