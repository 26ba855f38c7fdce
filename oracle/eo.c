/*
 * CPU oracle for the early-exit CNN hot path.  TEST INFRASTRUCTURE ONLY: it exists to
 * check the CUDA library and to be timed as a reported CPU baseline; no product path may
 * call it.  It shares no code, header, table or helper with the CUDA library.
 *
 * Everything here is the plain definition written out with fp64 accumulation and one loop
 * per index: no im2col, no tiling, no fused or reordered sums.  Activations are NHWC
 * float arrays, conv weights [Cout][kh][kw][Cin/groups], FC weights [K][C].
 *
 * What each function follows:
 *   eo_conv2d      a convolution layer is the matrix product of the Toeplitz (im2col) input
 *                  matrix R x P with the P x C weight matrix (paper Section II-C, Fig. "gemm",
 *                  Fig. 1 caption).  That product, element by element, is the direct
 *                  cross-correlation sum below with zero padding.  The folded-BN scale/bias,
 *                  residual add and ReLU/ReLU6 are the usual inference epilogue.
 *   eo_maxpool     3x3/s2 window maximum of the ResNet stem; padded taps are ignored.
 *   eo_exit_head   intermediate classifier with softmax top-1 as the confidence and one
 *                  threshold per exit (Section II-B; Section IV, Benchmarks).
 *   eo_compact     B_rem = B_act - B_exit samples stay, in order (Section III-B, Preemption
 *                  Mechanism; Algorithm 1).
 *   eo_refill      B_incr = min(N_Q, B_max - B_rem), B_merged = B_rem + B_incr
 *                  (Section III-B; Algorithm 1).
 *
 * Parity pins live in tests/test_oracle_pins.py (brute force, closed forms, library special
 * cases, the paper's scheduling-timeline example).  Exit-rate calibration built on top of
 * this file has no pin from the paper: "parity unpinned" for the calibrated scale factors.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

enum { EO_ACT_NONE = 0, EO_ACT_RELU = 1, EO_ACT_RELU6 = 2 };
enum { EO_ROUND_F32 = 0, EO_ROUND_BF16 = 1 };

/* Nearest bf16 (8 significant bits, 8 exponent bits), ties to even, from a double. */
double eo_round_bf16(double v) {
    if (v == 0.0 || isnan(v) || isinf(v)) return v;
    double a = fabs(v), r;
    int e;
    double m = frexp(a, &e);               /* a = m * 2^e, m in [0.5, 1) */
    if (e - 1 < -126) {                    /* below the smallest normal: fixed quantum 2^-133 */
        r = ldexp(nearbyint(ldexp(a, 133)), -133);
    } else {
        r = ldexp(nearbyint(ldexp(m, 8)), e - 8);   /* keep 8 significant bits */
        if (r > 3.3895313892515355e38) r = INFINITY; /* above the largest bf16 */
    }
    return v < 0 ? -r : r;
}

static double eo_round(double v, int mode) {
    return mode == EO_ROUND_BF16 ? eo_round_bf16(v) : (double)(float)v;
}

/* y[b,ho,wo,co] = act(scale[co] * sum_{r,s,ci} x[b, ho*st-pad_h+r, wo*st-pad_w+s, g*cpg+ci] * w[co,r,s,ci]
 *                     + bias[co] + residual[b,ho,wo,co]),  rounded once to the storage type.
 * Padding per axis: the factorised 1x7 / 7x1 convolutions of the paper's second benchmark network (Section IV,
 * Benchmarks: Inception-v3) keep the map size by padding only the axis the filter extends along. */
int eo_conv2d_hw(const float* x, int B, int H, int W, int Cin,
                 const float* w, int Cout, int kh, int kw, int stride, int pad_h, int pad_w, int groups,
                 const float* scale, const float* bias, const float* residual, int act, int rounding,
                 float* y) {
    if (groups < 1 || Cin % groups || Cout % groups) return 1;
    const int Ho = (H + 2 * pad_h - kh) / stride + 1, Wo = (W + 2 * pad_w - kw) / stride + 1;
    const int cpg = Cin / groups, opg = Cout / groups;
    if (Ho < 1 || Wo < 1) return 1;
    const long rows = (long)B * Ho;
#pragma omp parallel for schedule(dynamic, 1)
    for (long row = 0; row < rows; ++row) {
        const int b = (int)(row / Ho), ho = (int)(row % Ho);
        for (int wo = 0; wo < Wo; ++wo) {
            for (int co = 0; co < Cout; ++co) {
                const int g = co / opg;
                double acc = 0.0;
                for (int r = 0; r < kh; ++r) {
                    const int hi = ho * stride - pad_h + r;
                    if (hi < 0 || hi >= H) continue;
                    for (int s = 0; s < kw; ++s) {
                        const int wi = wo * stride - pad_w + s;
                        if (wi < 0 || wi >= W) continue;
                        const float* xp = x + (((size_t)b * H + hi) * W + wi) * Cin + (size_t)g * cpg;
                        const float* wp = w + (((size_t)co * kh + r) * kw + s) * cpg;
                        for (int ci = 0; ci < cpg; ++ci) acc += (double)xp[ci] * (double)wp[ci];
                    }
                }
                const size_t o = (((size_t)b * Ho + ho) * Wo + wo) * Cout + co;
                double v = (scale ? (double)scale[co] : 1.0) * acc + (bias ? (double)bias[co] : 0.0);
                if (residual) v += (double)residual[o];
                if (act == EO_ACT_RELU) v = v > 0.0 ? v : 0.0;
                else if (act == EO_ACT_RELU6) v = v > 0.0 ? (v < 6.0 ? v : 6.0) : 0.0;
                y[o] = (float)eo_round(v, rounding);
            }
        }
    }
    return 0;
}

/* The same padding on both axes. */
int eo_conv2d(const float* x, int B, int H, int W, int Cin,
              const float* w, int Cout, int kh, int kw, int stride, int pad, int groups,
              const float* scale, const float* bias, const float* residual, int act, int rounding,
              float* y) {
    return eo_conv2d_hw(x, B, H, W, Cin, w, Cout, kh, kw, stride, pad, pad, groups, scale, bias, residual, act, rounding, y);
}

/* Window maximum over the taps that fall inside the image. */
int eo_maxpool(const float* x, int B, int H, int W, int C, int k, int stride, int pad, float* y) {
    const int Ho = (H + 2 * pad - k) / stride + 1, Wo = (W + 2 * pad - k) / stride + 1;
    if (Ho < 1 || Wo < 1) return 1;
    for (int b = 0; b < B; ++b)
        for (int ho = 0; ho < Ho; ++ho)
            for (int wo = 0; wo < Wo; ++wo)
                for (int c = 0; c < C; ++c) {
                    double m = -INFINITY;
                    for (int r = 0; r < k; ++r) {
                        const int hi = ho * stride - pad + r;
                        if (hi < 0 || hi >= H) continue;
                        for (int s = 0; s < k; ++s) {
                            const int wi = wo * stride - pad + s;
                            if (wi < 0 || wi >= W) continue;
                            const double v = x[(((size_t)b * H + hi) * W + wi) * C + c];
                            if (v > m) m = v;
                        }
                    }
                    y[(((size_t)b * Ho + ho) * Wo + wo) * C + c] = (float)m;
                }
    return 0;
}

/* g[b,c] = mean_hw x[b,hw,c];  z[b,k] = sum_c Wfc[k,c] g[b,c] + bfc[k] (+ shift[b] on class shift_cls[b]);
 * conf[b] = max_k softmax(z[b,:]) = 1 / sum_k exp(z[b,k] - max z);  pred = lowest argmax;
 * exit[b] = always_exit or (float)conf >= (float)threshold  (the decision is taken in fp32, the
 * precision the CUDA library decides in; NaN never exits). */
int eo_exit_head(const float* x, int B, int HW, int C,
                 const float* wfc, const float* bfc, int K,
                 const float* shift, const int32_t* shift_cls,
                 float threshold, int always_exit,
                 double* gap, double* z, double* conf, int32_t* pred, uint8_t* exit_mask) {
    for (int b = 0; b < B; ++b) {
        double* g = gap + (size_t)b * C;
        for (int c = 0; c < C; ++c) {
            double s = 0.0;
            for (int p = 0; p < HW; ++p) s += (double)x[((size_t)b * HW + p) * C + c];
            g[c] = s / (double)HW;
        }
        double* zb = z + (size_t)b * K;
        for (int k = 0; k < K; ++k) {
            double s = 0.0;
            for (int c = 0; c < C; ++c) s += (double)wfc[(size_t)k * C + c] * g[c];
            zb[k] = s + (bfc ? (double)bfc[k] : 0.0);
        }
        if (shift && shift_cls && shift_cls[b] >= 0 && shift_cls[b] < K) zb[shift_cls[b]] += (double)shift[b];
        int arg = 0;
        for (int k = 1; k < K; ++k)
            if (zb[k] > zb[arg]) arg = k;
        double den = 0.0;
        for (int k = 0; k < K; ++k) den += exp(zb[k] - zb[arg]);
        conf[b] = 1.0 / den;
        pred[b] = arg;
        exit_mask[b] = (uint8_t)(always_exit ? 1 : ((float)conf[b] >= threshold ? 1 : 0));
    }
    return 0;
}

/* Samples with exit_mask == 0 move to the front, order kept.  Returns n_surv. */
int eo_compact(const uint8_t* exit_mask, int B, const float* feat, size_t elems_per_sample,
               const int32_t* ids, int32_t* surv_idx, float* feat_out, int32_t* ids_out) {
    int n = 0;
    for (int b = 0; b < B; ++b) {
        if (exit_mask[b]) continue;
        surv_idx[n] = b;
        if (feat && feat_out) memcpy(feat_out + (size_t)n * elems_per_sample, feat + (size_t)b * elems_per_sample, elems_per_sample * sizeof(float));
        if (ids && ids_out) ids_out[n] = ids[b];
        ++n;
    }
    return n;
}

/* batch <- survivors ++ arrivals[0 : n_acc], n_acc = min(n_arr, max_batch - n_surv).  Returns n_acc. */
int eo_refill(float* batch_feat, int32_t* batch_ids, int n_surv, size_t elems_per_sample,
              const float* arr_feat, const int32_t* arr_ids, int n_arr, int max_batch) {
    int slack = max_batch - n_surv;
    if (slack < 0) return -1;
    int n_acc = n_arr < slack ? n_arr : slack;
    for (int j = 0; j < n_acc; ++j) {
        memcpy(batch_feat + (size_t)(n_surv + j) * elems_per_sample, arr_feat + (size_t)j * elems_per_sample, elems_per_sample * sizeof(float));
        if (batch_ids && arr_ids) batch_ids[n_surv + j] = arr_ids[j];
    }
    return n_acc;
}
