/*
 * TEST INFRASTRUCTURE ONLY -- CPU oracle for the forward layers of a CNN.
 *
 * Plain, slow, direct implementations written from the paper's definitions:
 *   - convolution layer:  Section II (each output-feature-map pixel is the sum,
 *     over numInputLayers, of a KxK kernel applied to the input window, the
 *     window sliding by stride S) and the sequential loop nest described in
 *     Section III (Fig. 2 prose: one outer loop over output layers around a
 *     3-D convolution of the input with one filter bank).
 *   - pooling and softmax: Section III-E.
 *
 * Layouts are the paper's default row-major order (Eq. 5):
 *   activations [batch][layer][row][col], kernels [outLayer][inLayer][K][K].
 * Storage is float; every accumulation is done in double and rounded to float
 * once, when the element is stored.
 *
 * Only tests, the smoke check and the benchmark's CPU-baseline leg may use
 * this file.  It shares nothing with the CUDA library.
 */
#include <math.h>
#include <stddef.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_max_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Output extent of a sliding window: (H + 2*pad - K) / S + 1, integer division. */
int oracle_out_extent(int H, int K, int S, int pad)
{
    return (H + 2 * pad - K) / S + 1;
}

/*
 * Convolution layer (Section II; Section III, Fig. 2 prose).
 *   out[n][m][h][w] = act( bias[m] + sum_{c,i,j} in[n][c][h*S+i-pad][w*S+j-pad] * ker[m][c][i][j] )
 * Window positions that fall outside the input contribute zero (zero padding).
 * The kernel is applied as a dot product with the window: no flip.
 * act is max(.,0) when relu != 0, identity otherwise.  bias may be NULL (zero).
 */
void oracle_conv2d(const float *in, const float *ker, const float *bias, float *out,
                   int batch, int numInputLayers, int H, int W,
                   int numOutputLayers, int K, int S, int pad, int relu)
{
    const int outH = oracle_out_extent(H, K, S, pad);
    const int outW = oracle_out_extent(W, K, S, pad);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < batch; ++n) {
        for (int m = 0; m < numOutputLayers; ++m) {            /* loop #1: output layers */
            for (int h = 0; h < outH; ++h) {
                for (int w = 0; w < outW; ++w) {
                    double acc = bias ? (double)bias[m] : 0.0;
                    for (int c = 0; c < numInputLayers; ++c) {
                        for (int i = 0; i < K; ++i) {
                            const int y = h * S + i - pad;
                            if (y < 0 || y >= H) continue;
                            for (int j = 0; j < K; ++j) {
                                const int x = w * S + j - pad;
                                if (x < 0 || x >= W) continue;
                                const double a = in[(((size_t)n * numInputLayers + c) * H + y) * W + x];
                                const double k = ker[(((size_t)m * numInputLayers + c) * K + i) * K + j];
                                acc += a * k;
                            }
                        }
                    }
                    if (relu && acc < 0.0) acc = 0.0;
                    out[(((size_t)n * numOutputLayers + m) * outH + h) * outW + w] = (float)acc;
                }
            }
        }
    }
}

/*
 * Max pooling (Section III-E): maximum over a KxK window slid by S, no padding,
 * output extent (H - K) / S + 1.
 */
void oracle_maxpool(const float *in, float *out, int batch, int layers, int H, int W, int K, int S)
{
    const int outH = oracle_out_extent(H, K, S, 0);
    const int outW = oracle_out_extent(W, K, S, 0);
    #pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < batch; ++n) {
        for (int c = 0; c < layers; ++c) {
            const float *src = in + ((size_t)n * layers + c) * H * W;
            float *dst = out + ((size_t)n * layers + c) * outH * outW;
            for (int h = 0; h < outH; ++h) {
                for (int w = 0; w < outW; ++w) {
                    float best = src[(size_t)(h * S) * W + (w * S)];
                    for (int i = 0; i < K; ++i)
                        for (int j = 0; j < K; ++j) {
                            const float v = src[(size_t)(h * S + i) * W + (w * S + j)];
                            if (v > best) best = v;
                        }
                    dst[(size_t)h * outW + w] = best;
                }
            }
        }
    }
}

/* Average pooling over the whole map (Section III-E): z[n][c] = mean over rows and columns. */
void oracle_global_avgpool(const float *in, float *out, int batch, int layers, int H, int W)
{
    for (int n = 0; n < batch; ++n)
        for (int c = 0; c < layers; ++c) {
            const float *src = in + ((size_t)n * layers + c) * H * W;
            double s = 0.0;
            for (int p = 0; p < H * W; ++p) s += (double)src[p];
            out[(size_t)n * layers + c] = (float)(s / (double)(H * W));
        }
}

/* Softmax over the class scores of each image (Section III-E), max-subtracted. */
void oracle_softmax(const float *z, float *p, int batch, int classes)
{
    for (int n = 0; n < batch; ++n) {
        const float *zi = z + (size_t)n * classes;
        float *pi = p + (size_t)n * classes;
        double zmax = (double)zi[0];
        for (int k = 1; k < classes; ++k) if ((double)zi[k] > zmax) zmax = (double)zi[k];
        double sum = 0.0;
        for (int k = 0; k < classes; ++k) sum += exp((double)zi[k] - zmax);
        for (int k = 0; k < classes; ++k) pi[k] = (float)(exp((double)zi[k] - zmax) / sum);
    }
}
