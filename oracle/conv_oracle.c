/*
 * CPU oracle for the convolution-layer forward pass.  TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, obviously-correct statement of what the GPU library must compute.
 * It is used by the test-suite, by the smoke check and by the benchmark's CPU-baseline leg and
 * by nothing else; the product (the CUDA library and its Python binding) never links, imports
 * or calls it, and it shares no code with the CUDA path.
 *
 * Everything is fp64.  Inputs arrive as doubles (the caller widens the fp32 arrays exactly),
 * accumulation is in double in the fixed order c, r, s, and the result is stored as double.
 * There is no blocking, no im2col matrix, no vector intrinsic and no reordering: the loops are
 * the definition, so that they can be checked against the paper by eye.  OpenMP only spreads
 * independent (n, k) output planes over host threads; it never changes a summation order.
 *
 * Paper passages followed (Section 2, "Introduction to CNN Computations"):
 *   - out = conv(in, filts); one filter slice per output channel computes one output plane;
 *   - output extent  1 + (in_X - KSZ) / stride  per spatial dimension, after optional padding of
 *     the input with zeros;
 *   - the window of `in` that feeds out[oc, oy, ox] starts at (oy*stride, ox*stride) and spans
 *     KSZ x KSZ pixels over all input channels;
 *   - the output value is the sum of the element-wise product of that window and the filter
 *     slice (no flip: a cross-correlation);
 *   - results for different images of a batch are independent;
 *   - the activation ReLU = max(0, x) is applied to each output value after the sum.
 * The paper leaves the bias out of its discussion; the reading taken here is a per-output-channel
 * constant added before the activation.  Non-divisible extents take the floor.
 *
 * Parity pins: every function below is pinned by tests/test_oracle_pins.py (worked example of the
 * paper, hand-computed cases, closed forms, identities, brute-force im2col and library
 * cross-checks).  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>

/* Output extent of one spatial dimension (Section 2: out_X = 1 + (in_X - KSZ)/stride, applied to
 * the padded extent, floor division).  Returns 0 when the padded input is smaller than the window. */
int oracle_conv_out_dim(int in_dim, int ksz, int stride, int pad)
{
    int padded = in_dim + 2 * pad;
    if (in_dim <= 0 || ksz <= 0 || stride <= 0 || pad < 0 || padded < ksz) return 0;
    return 1 + (padded - ksz) / stride;
}

/*
 * in   [N][C][H][W]      filt [K][C][R][S]      bias [K] or NULL      out [N][K][P][Q]
 * All dense, row-major, double.  Returns 0, or -1 on an invalid shape.
 */
int oracle_conv_fwd_f64(const double *in, const double *filt, const double *bias, double *out,
                        int N, int C, int H, int W, int K, int R, int S,
                        int stride, int pad, int relu)
{
    const int P = oracle_conv_out_dim(H, R, stride, pad);
    const int Q = oracle_conv_out_dim(W, S, stride, pad);
    if (N <= 0 || C <= 0 || K <= 0 || P <= 0 || Q <= 0 || !in || !filt || !out) return -1;

    long long nk;
#pragma omp parallel for schedule(dynamic, 1)
    for (nk = 0; nk < (long long)N * K; ++nk) {
        const int n = (int)(nk / K);
        const int k = (int)(nk % K);
        for (int p = 0; p < P; ++p) {
            for (int q = 0; q < Q; ++q) {
                double acc = bias ? bias[k] : 0.0;
                for (int c = 0; c < C; ++c) {
                    for (int r = 0; r < R; ++r) {
                        const int y = p * stride + r - pad;      /* row in the unpadded input */
                        if (y < 0 || y >= H) continue;           /* padding rows are zeros     */
                        for (int s = 0; s < S; ++s) {
                            const int x = q * stride + s - pad;
                            if (x < 0 || x >= W) continue;
                            acc += in[(((size_t)n * C + c) * H + y) * W + x] *
                                   filt[(((size_t)k * C + c) * R + r) * S + s];
                        }
                    }
                }
                if (relu && !(acc > 0.0)) acc = 0.0;
                out[(((size_t)n * K + k) * P + p) * Q + q] = acc;
            }
        }
    }
    return 0;
}

/*
 * Max-pooling over ksz x ksz windows with the given stride, no padding, floor output extent
 * (the pooling between the layers of the AlexNet-shaped stack; the paper names pooling as a
 * deployment operation without specifying it further, so the common definition is taken).
 * in [N][C][H][W] -> out [N][C][1+(H-ksz)/stride][1+(W-ksz)/stride].
 */
int oracle_maxpool_fwd_f64(const double *in, double *out, int N, int C, int H, int W,
                           int ksz, int stride)
{
    const int P = oracle_conv_out_dim(H, ksz, stride, 0);
    const int Q = oracle_conv_out_dim(W, ksz, stride, 0);
    if (N <= 0 || C <= 0 || P <= 0 || Q <= 0 || !in || !out) return -1;
    long long nc;
#pragma omp parallel for schedule(static)
    for (nc = 0; nc < (long long)N * C; ++nc) {
        const double *src = in + (size_t)nc * H * W;
        double *dst = out + (size_t)nc * P * Q;
        for (int p = 0; p < P; ++p)
            for (int q = 0; q < Q; ++q) {
                double best = src[(size_t)(p * stride) * W + q * stride];
                for (int r = 0; r < ksz; ++r)
                    for (int s = 0; s < ksz; ++s) {
                        const double v = src[(size_t)(p * stride + r) * W + q * stride + s];
                        if (v > best) best = v;
                    }
                dst[(size_t)p * Q + q] = best;
            }
    }
    return 0;
}

/* Multiply-accumulates of one layer: one per (output point, filter element). */
long long oracle_conv_macs(int N, int C, int H, int W, int K, int R, int S, int stride, int pad)
{
    const long long P = oracle_conv_out_dim(H, R, stride, pad);
    const long long Q = oracle_conv_out_dim(W, S, stride, pad);
    return (long long)N * K * P * Q * C * R * S;
}

/* Compulsory bytes of one fp32 layer: every tensor touched exactly once (in, filt, bias, out). */
long long oracle_conv_min_bytes(int N, int C, int H, int W, int K, int R, int S, int stride, int pad)
{
    const long long P = oracle_conv_out_dim(H, R, stride, pad);
    const long long Q = oracle_conv_out_dim(W, S, stride, pad);
    return 4LL * ((long long)N * C * H * W + (long long)K * C * R * S + K + (long long)N * K * P * Q);
}

/* Arithmetic intensity of SGEMM, Section 4: AI = 2MNK / 4(MN + MK + KN), FLOPs per byte. */
double oracle_sgemm_ai(long long M, long long N, long long K)
{
    return (2.0 * (double)M * (double)N * (double)K) /
           (4.0 * ((double)M * N + (double)M * K + (double)K * N));
}

/*
 * SGEMM, Section 4 (the paper's warm-up; Table 1): C[i][j] = sum over k of A[i][k] * B[k][j], all row-major.
 * The definition written out: one fp64 accumulator per element, k ascending.  OpenMP over rows only.
 * Returns 0 on success, 1 on invalid arguments.
 */
int oracle_sgemm_f64(const double* A, const double* B, double* C, int M, int N, int K)
{
    if (!A || !B || !C || M <= 0 || N <= 0 || K <= 0) return 1;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < M; ++i)
        for (int j = 0; j < N; ++j) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += A[(size_t)i * K + k] * B[(size_t)k * N + j];
            C[(size_t)i * N + j] = acc;
        }
    return 0;
}

/*
 * Softmax over the last dimension (Section 2 lists it with convolution and pooling as the operations deployment
 * needs; the paper does not analyse it): out[r][j] = exp(in[r][j]) / sum over i of exp(in[r][i]).
 * The definition written out in fp64; the row maximum is subtracted first, which changes no quotient and keeps exp
 * inside its range.  Returns 0 on success, 1 on invalid arguments.
 */
int oracle_softmax_f64(const double* in, double* out, int rows, int cols)
{
    if (!in || !out || rows <= 0 || cols <= 0) return 1;
    for (int r = 0; r < rows; ++r) {
        const double* x = in + (size_t)r * cols;
        double* y = out + (size_t)r * cols;
        double mx = x[0];
        for (int j = 1; j < cols; ++j) if (x[j] > mx) mx = x[j];
        double sum = 0.0;
        for (int j = 0; j < cols; ++j) { y[j] = exp(x[j] - mx); sum += y[j]; }
        for (int j = 0; j < cols; ++j) y[j] /= sum;
    }
    return 0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
