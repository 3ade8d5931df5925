/*
 * Oracle (test infrastructure): the policies (paper Section 4, "Exploring Novel
 * Policy Architectures": get_actions maps task states and a member's parameters to
 * actions; Section 3 names an MLP-controlled cart-pole and a ConvNet classifier).
 * Both policies are stateless.  Parameter order and layer shapes are this
 * repository's reading; the paper gives none.
 */
#include "oracle.h"
#include <math.h>
#include <string.h>
#include <stdlib.h>

uint32_t oracle_mlp_param_count(uint32_t n_layers, const uint32_t* sizes)
{
    uint32_t n = 0;
    for (uint32_t l = 0; l < n_layers; ++l) n += sizes[l + 1] * sizes[l] + sizes[l + 1];
    return n;
}

void oracle_mlp_forward(const double* params, uint32_t n_layers, const uint32_t* sizes,
                        const double* x, double* y, double action_scale)
{
    double in[1024], out[1024];
    for (uint32_t k = 0; k < sizes[0]; ++k) in[k] = x[k];
    const double* p = params;
    for (uint32_t l = 0; l < n_layers; ++l) {
        uint32_t n_in = sizes[l], n_out = sizes[l + 1];
        const double* W = p;
        const double* b = p + (size_t)n_out * n_in;
        for (uint32_t i = 0; i < n_out; ++i) {
            double acc = b[i];
            for (uint32_t k = 0; k < n_in; ++k) acc += W[(size_t)i * n_in + k] * in[k];
            out[i] = tanh(acc);
        }
        for (uint32_t i = 0; i < n_out; ++i) in[i] = out[i];
        p += (size_t)n_out * n_in + n_out;
    }
    for (uint32_t i = 0; i < sizes[n_layers]; ++i) y[i] = action_scale * in[i];
}

/* ---- convolutional policy ----------------------------------------------------- */

float oracle_bf16_round(float x)
{
    /* round to nearest even onto the upper 16 bits of the fp32 pattern */
    uint32_t b;
    memcpy(&b, &x, 4);
    if ((b & 0x7F800000u) == 0x7F800000u) return x;          /* inf / nan unchanged */
    uint32_t lsb = (b >> 16) & 1u;
    b += 0x7FFFu + lsb;
    b &= 0xFFFF0000u;
    float y;
    memcpy(&y, &b, 4);
    return y;
}

/* an operand of a contraction: rounded to bf16 (through fp32) in the bf16 reading */
static double operand(double x, int bf16) { return bf16 ? (double)oracle_bf16_round((float)x) : x; }

enum { C1 = 8, C2 = 16, KS = 5, IMG = 28, O1 = 24, Q1 = 12, O2 = 8, Q2 = 4, NCLS = 10 };

void oracle_cnn_logits(const float* params, const float* image, int bf16, double logits[10])
{
    const float* w1  = params;                       /* [8][1][5][5]  */
    const float* b1  = w1 + C1 * KS * KS;            /* [8]           */
    const float* w2  = b1 + C1;                      /* [16][8][5][5] */
    const float* b2  = w2 + C2 * C1 * KS * KS;       /* [16]          */
    const float* wfc = b2 + C2;                      /* [10][256]     */
    const float* bfc = wfc + NCLS * C2 * Q2 * Q2;    /* [10]          */

    double conv1[C1][O1][O1];
    double pool1[C1][Q1][Q1];
    double conv2[C2][O2][O2];
    double pool2[C2][Q2][Q2];

    /* conv 1 -> 8, 5x5, stride 1, no padding (cross-correlation), + bias, ReLU */
    for (int oc = 0; oc < C1; ++oc)
        for (int y = 0; y < O1; ++y)
            for (int x = 0; x < O1; ++x) {
                double acc = 0.0;
                for (int kh = 0; kh < KS; ++kh)
                    for (int kw = 0; kw < KS; ++kw)
                        acc += operand(w1[(oc * KS + kh) * KS + kw], bf16) *
                               operand(image[(y + kh) * IMG + (x + kw)], bf16);
                acc += (double)b1[oc];
                conv1[oc][y][x] = acc > 0.0 ? acc : 0.0;
            }
    /* 2x2 max pool, stride 2 */
    for (int c = 0; c < C1; ++c)
        for (int y = 0; y < Q1; ++y)
            for (int x = 0; x < Q1; ++x) {
                double m = conv1[c][2 * y][2 * x];
                if (conv1[c][2 * y][2 * x + 1] > m) m = conv1[c][2 * y][2 * x + 1];
                if (conv1[c][2 * y + 1][2 * x] > m) m = conv1[c][2 * y + 1][2 * x];
                if (conv1[c][2 * y + 1][2 * x + 1] > m) m = conv1[c][2 * y + 1][2 * x + 1];
                pool1[c][y][x] = m;
            }
    /* conv 8 -> 16, 5x5, + bias, ReLU */
    for (int oc = 0; oc < C2; ++oc)
        for (int y = 0; y < O2; ++y)
            for (int x = 0; x < O2; ++x) {
                double acc = 0.0;
                for (int ic = 0; ic < C1; ++ic)
                    for (int kh = 0; kh < KS; ++kh)
                        for (int kw = 0; kw < KS; ++kw)
                            acc += operand(w2[((oc * C1 + ic) * KS + kh) * KS + kw], bf16) *
                                   operand(pool1[ic][y + kh][x + kw], bf16);
                acc += (double)b2[oc];
                conv2[oc][y][x] = acc > 0.0 ? acc : 0.0;
            }
    for (int c = 0; c < C2; ++c)
        for (int y = 0; y < Q2; ++y)
            for (int x = 0; x < Q2; ++x) {
                double m = conv2[c][2 * y][2 * x];
                if (conv2[c][2 * y][2 * x + 1] > m) m = conv2[c][2 * y][2 * x + 1];
                if (conv2[c][2 * y + 1][2 * x] > m) m = conv2[c][2 * y + 1][2 * x];
                if (conv2[c][2 * y + 1][2 * x + 1] > m) m = conv2[c][2 * y + 1][2 * x + 1];
                pool2[c][y][x] = m;
            }
    /* linear 256 -> 10 on the (channel, row, column) flattening */
    for (int o = 0; o < NCLS; ++o) {
        double acc = 0.0;
        for (int c = 0; c < C2; ++c)
            for (int y = 0; y < Q2; ++y)
                for (int x = 0; x < Q2; ++x)
                    acc += operand(wfc[o * (C2 * Q2 * Q2) + (c * Q2 + y) * Q2 + x], bf16) *
                           operand(pool2[c][y][x], bf16);
        logits[o] = acc + (double)bfc[o];
    }
}

double oracle_cnn_fitness(const float* params, const float* images, const int32_t* labels,
                          uint32_t B, int bf16)
{
    double loss = 0.0;
    for (uint32_t i = 0; i < B; ++i) {
        double logits[NCLS];
        oracle_cnn_logits(params, images + (size_t)i * IMG * IMG, bf16, logits);
        double mx = logits[0];
        for (int o = 1; o < NCLS; ++o) if (logits[o] > mx) mx = logits[o];
        double se = 0.0;
        for (int o = 0; o < NCLS; ++o) se += exp(logits[o] - mx);
        loss += (mx + log(se)) - logits[labels[i]];
    }
    return -loss / (double)B;
}
