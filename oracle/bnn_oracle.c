/*
 * CPU oracle for the forward pass of a feed-forward DNN with binary (+-1) weights and
 * activations (Lu, arXiv 1706.09453).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is deliberately plain and slow: every quantity is the
 * paper's definition written out as nested loops.  +-1 dot products are integer sums of
 * products over decoded int8 values (no XOR, no popcount); real-valued layers and the
 * log-softmax are evaluated in double.  It shares no code with the CUDA library and must
 * never be called from the product path.  All pointers are HOST pointers.
 *
 * Conventions (the paper fixes none for storage; these are this project's):
 *   bit = 1 <=> +1, bit = 0 <=> -1 (activations of a (0,1) network: bit = the value itself);
 *   element k of a row is bit k%32 of 32-bit word k/32;
 *   bits at positions >= K are zero.  Row pitches (ld*) are in elements of the array type.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -fPIC -shared bnn_oracle.c -o libbnn_oracle.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define SIGN_ZERO_POS 0 /* Sign(0) = +1 */
#define SIGN_ZERO_NEG 1 /* Sign(0) = -1: Eq. 3 as printed (+1 if x > 0, -1 otherwise) */

#define ACT_NONE 0
#define ACT_SIGN 1
#define ACT_HARDTANH 2
#define ACT_SIGMOID 3  /* the hidden units of the paper's real-valued layers (Section 3) */

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Eq. 3.  NaN compares false in both modes and therefore maps to -1. */
int oracle_sign_f32(float x, int mode) {
    if (mode == SIGN_ZERO_NEG) return x > 0.0f ? 1 : -1;
    return x >= 0.0f ? 1 : -1;
}

static int sign_f64(double x, int mode) {
    if (mode == SIGN_ZERO_NEG) return x > 0.0 ? 1 : -1;
    return x >= 0.0 ? 1 : -1;
}

/* Binarise (Eq. 3) a real matrix and store one bit per element. */
void oracle_sign_pack(const float* X, long M, long K, long ldx, uint32_t* P, long ldp, int mode) {
    for (long m = 0; m < M; ++m) {
        for (long w = 0; w < ldp; ++w) P[m * ldp + w] = 0u;
        for (long k = 0; k < K; ++k) {
            if (oracle_sign_f32(X[m * ldx + k], mode) == 1)
                P[m * ldp + k / 32] |= (uint32_t)1 << (k % 32);
        }
    }
}

/* Decode a packed plane to +-1 values. */
void oracle_unpack_pm1(const uint32_t* P, long ldp, long M, long K, int8_t* S) {
    for (long m = 0; m < M; ++m)
        for (long k = 0; k < K; ++k)
            S[m * K + k] = ((P[m * ldp + k / 32] >> (k % 32)) & 1u) ? 1 : -1;
}

/* Decode a packed plane to (0,1) values: the binary pair the paper compares with (-1,+1)
 * for activations (Section 3.2, Table 3; Section 3.3, Table 4). */
void oracle_unpack_01(const uint32_t* P, long ldp, long M, long K, int8_t* S) {
    for (long m = 0; m < M; ++m)
        for (long k = 0; k < K; ++k)
            S[m * K + k] = (int8_t)((P[m * ldp + k / 32] >> (k % 32)) & 1u);
}

/*
 * Binary weights in {-1,+1} against binary activations in {0,1} (Section 3.2: "(0,1) for
 * binary activations"): d[m][n] = sum_k h[m][k] * w[n][k].  Exact integer arithmetic.
 */
void oracle_gemm01(const uint32_t* Hp, long ldhp, const uint32_t* Wp, long ldwp,
                   long M, long N, long K, int32_t* D, long ldd) {
    int8_t* h = (int8_t*)malloc((size_t)M * K);
    int8_t* w = (int8_t*)malloc((size_t)N * K);
    oracle_unpack_01(Hp, ldhp, M, K, h);
    oracle_unpack_pm1(Wp, ldwp, N, K, w);
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long n = 0; n < N; ++n) {
            int32_t s = 0;
            for (long k = 0; k < K; ++k) s += (int32_t)h[m * K + k] * (int32_t)w[n * K + k];
            D[m * ldd + n] = s;
        }
    }
    free(h);
    free(w);
}

/*
 * Binary weights and binary activations (Section 2.3): the pre-activation without bias,
 * d[m][n] = sum_k a[m][k] * w[n][k], with a, w in {-1,+1}.  Exact integer arithmetic.
 */
void oracle_xnor_gemm(const uint32_t* Ap, long ldap, const uint32_t* Wp, long ldwp,
                      long M, long N, long K, int32_t* D, long ldd) {
    int8_t* a = (int8_t*)malloc((size_t)M * K);
    int8_t* w = (int8_t*)malloc((size_t)N * K);
    oracle_unpack_pm1(Ap, ldap, M, K, a);
    oracle_unpack_pm1(Wp, ldwp, N, K, w);
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long n = 0; n < N; ++n) {
            int32_t s = 0;
            for (long k = 0; k < K; ++k) s += (int32_t)a[m * K + k] * (int32_t)w[n * K + k];
            D[m * ldd + n] = s;
        }
    }
    free(a);
    free(w);
}

/*
 * Hidden binary layer, after the dot product: h = Sign(scale*d + shift) (Eq. 1-2 with
 * f = Sign; Algorithm 2 forward).  The paper has only a bias (scale = 1); the per-unit
 * scale generalises it.  The affine is ONE fused multiply-add in fp32 (single rounding),
 * which is what decides the bit when the value is near zero.
 * scale == NULL means 1, shift == NULL means 0.  Y (optional) receives the fp32 value.
 */
void oracle_affine_sign_pack_i32(const int32_t* D, long ldd, long M, long N,
                                 const float* scale, const float* shift, int mode,
                                 uint32_t* P, long ldp, float* Y, long ldy) {
    for (long m = 0; m < M; ++m) {
        for (long w = 0; w < ldp; ++w) P[m * ldp + w] = 0u;
        for (long n = 0; n < N; ++n) {
            float s = scale ? scale[n] : 1.0f;
            float b = shift ? shift[n] : 0.0f;
            float y = fmaf(s, (float)D[m * ldd + n], b);
            if (Y) Y[m * ldy + n] = y;
            if (oracle_sign_f32(y, mode) == 1) P[m * ldp + n / 32] |= (uint32_t)1 << (n % 32);
        }
    }
}

/*
 * A binary layer whose output stays real-valued: h = Sigmoid(scale*d + shift), the last hidden
 * layer of the paper's best systems (Table 2: Sigmoid on the first and last hidden layer, binary
 * in between).  The affine is the same single fp32 fused multiply-add as in the Sign layers; the
 * Sigmoid of that fp32 value is evaluated in double.  Yhat (optional) receives the fp32 value.
 */
void oracle_affine_sigmoid_i32(const int32_t* D, long ldd, long M, long N,
                               const float* scale, const float* shift,
                               double* H, long ldh, float* Yhat, long ldy) {
    for (long m = 0; m < M; ++m)
        for (long n = 0; n < N; ++n) {
            float s = scale ? scale[n] : 1.0f;
            float b = shift ? shift[n] : 0.0f;
            float y = fmaf(s, (float)D[m * ldd + n], b);
            if (Yhat) Yhat[m * ldy + n] = y;
            H[m * ldh + n] = 1.0 / (1.0 + exp(-(double)y));
        }
}

/*
 * Binary weights against real-valued activations (Algorithm 1 forward, without the bias):
 * y[m][n] = sum_k w^b[n][k] * x[m][k], w^b in {-1,+1}, accumulated in double.
 * sumabs[m] (optional) = sum_k |x[m][k]|, the scale of the comparison tolerance.
 */
void oracle_signw_gemm(const float* X, long ldx, const uint32_t* Wp, long ldwp,
                       long M, long N, long K, double* Y, long ldy, double* sumabs) {
    int8_t* w = (int8_t*)malloc((size_t)N * K);
    oracle_unpack_pm1(Wp, ldwp, N, K, w);
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long n = 0; n < N; ++n) {
            double s = 0.0;
            for (long k = 0; k < K; ++k) s += (double)w[n * K + k] * (double)X[m * ldx + k];
            Y[m * ldy + n] = s;
        }
        if (sumabs) {
            double t = 0.0;
            for (long k = 0; k < K; ++k) t += fabs((double)X[m * ldx + k]);
            sumabs[m] = t;
        }
    }
    free(w);
}

/*
 * Per-unit affine and activation on a real-valued pre-activation (Eq. 1-2), in double:
 * yhat = scale*y + shift; then Sign (-> bits P and +-1 in H), clamp to [-1,1] (H), or
 * nothing (H = yhat).  Yhat (optional) receives the value before the activation.
 */
void oracle_affine_act_f64(const double* Y, long ldy, long M, long N,
                           const float* scale, const float* shift, int act, int mode,
                           double* Yhat, long ldyh, double* H, long ldh,
                           uint32_t* P, long ldp) {
    for (long m = 0; m < M; ++m) {
        if (P) for (long w = 0; w < ldp; ++w) P[m * ldp + w] = 0u;
        for (long n = 0; n < N; ++n) {
            double s = scale ? (double)scale[n] : 1.0;
            double b = shift ? (double)shift[n] : 0.0;
            double v = s * Y[m * ldy + n] + b;
            if (Yhat) Yhat[m * ldyh + n] = v;
            double h = v;
            if (act == ACT_SIGN) {
                int sg = sign_f64(v, mode);
                h = (double)sg;
                if (P && sg == 1) P[m * ldp + n / 32] |= (uint32_t)1 << (n % 32);
            } else if (act == ACT_HARDTANH) {
                h = v < -1.0 ? -1.0 : (v > 1.0 ? 1.0 : v);
            } else if (act == ACT_SIGMOID) {
                h = 1.0 / (1.0 + exp(-v));
            }
            if (H) H[m * ldh + n] = h;
        }
    }
}

/*
 * Real-valued top layer (Section 2.3: the Softmax layer keeps real weights) on +-1
 * activations given as bits: z[m][c] = sum_n Wout[c][n]*h[m][n] + b[c], in double.
 */
void oracle_real_gemm_bits(const uint32_t* Hp, long ldhp, const float* Wout, long ldw,
                           const float* b, long M, long C, long H, double* Z, long ldz) {
    int8_t* h = (int8_t*)malloc((size_t)M * H);
    oracle_unpack_pm1(Hp, ldhp, M, H, h);
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long c = 0; c < C; ++c) {
            double s = 0.0;
            for (long n = 0; n < H; ++n) s += (double)Wout[c * ldw + n] * (double)h[m * H + n];
            Z[m * ldz + c] = s + (b ? (double)b[c] : 0.0);
        }
    }
    free(h);
}

/* The same top layer on (0,1) activations given as bits (Section 3.2). */
void oracle_real_gemm_bits01(const uint32_t* Hp, long ldhp, const float* Wout, long ldw,
                             const float* b, long M, long C, long H, double* Z, long ldz) {
    int8_t* h = (int8_t*)malloc((size_t)M * H);
    oracle_unpack_01(Hp, ldhp, M, H, h);
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long c = 0; c < C; ++c) {
            double s = 0.0;
            for (long n = 0; n < H; ++n) s += (double)Wout[c * ldw + n] * (double)h[m * H + n];
            Z[m * ldz + c] = s + (b ? (double)b[c] : 0.0);
        }
    }
    free(h);
}

/* Same top layer on real-valued activations (binary-weights-only networks). */
void oracle_real_gemm_f32(const float* Hf, long ldh, const float* Wout, long ldw,
                          const float* b, long M, long C, long H, double* Z, long ldz) {
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        for (long c = 0; c < C; ++c) {
            double s = 0.0;
            for (long n = 0; n < H; ++n) s += (double)Wout[c * ldw + n] * (double)Hf[m * ldh + n];
            Z[m * ldz + c] = s + (b ? (double)b[c] : 0.0);
        }
    }
}

/* log of the Softmax of Algorithm 2's top layer: z - max - log(sum exp(z - max)). */
void oracle_log_softmax(const double* Z, long ldz, long M, long C, double* LP, long ldlp) {
#pragma omp parallel for schedule(static)
    for (long m = 0; m < M; ++m) {
        double mx = Z[m * ldz];
        for (long c = 1; c < C; ++c) if (Z[m * ldz + c] > mx) mx = Z[m * ldz + c];
        double s = 0.0;
        for (long c = 0; c < C; ++c) s += exp(Z[m * ldz + c] - mx);
        double lse = mx + log(s);
        for (long c = 0; c < C; ++c) LP[m * ldlp + c] = Z[m * ldz + c] - lse;
    }
}
