/*
 * CPU oracle (test infrastructure only): the sequence-to-sequence addition task with an LSTM
 * encoder-decoder policy (paper Section 3, "Seq2Seq Learning": the query spells the addition of
 * two random integers padded with leading zeros, e.g. "012+345=", and the policy must spell the
 * sum; an LSTM-based seq2seq model is evolved).
 *
 * The paper fixes the task in words only; the concrete conventions below are this repository's
 * readings: vocabulary '0'..'9' -> 0..9, '+' -> 10, '=' -> 11; the encoder reads "a+b"
 * (2 nd + 1 tokens), the decoder is fed '=' and then the true answer digits (teacher forcing) and
 * must produce the nd + 1 digits of the sum, most significant first; one LSTM layer each for
 * encoder and decoder (gate order input, forget, cell, output), the decoder starting from the
 * encoder's final (h, c); a linear read-out to the 12 tokens; fitness = minus the mean
 * cross-entropy over all answer positions of the batch.
 *
 * Flat parameter order: enc.Wx[4h][12], enc.Wh[4h][h], enc.b[4h], dec.Wx, dec.Wh, dec.b,
 * out.W[12][h], out.b[12].
 *
 * bf16 reading: a cell's pre-activation is ONE contraction, [Wh | Wx | b] . [h; onehot(token); 1],
 * and the read-out is another, out.W . h; the operands of both (Wh, Wx, b, out.W and the hidden
 * state; the one-hot vector and the 1 are exact) are rounded to bf16.  The read-out bias, the
 * gates, the cell state and the softmax are not rounded.
 */
#include "oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

enum { VOCAB = 12, TOK_PLUS = 10, TOK_EQ = 11 };

static double operand(double x, int bf16) { return bf16 ? (double)oracle_bf16_round((float)x) : x; }
static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

uint32_t oracle_seq2seq_param_count(uint32_t h)
{
    return 2u * (4u * h * VOCAB + 4u * h * h + 4u * h) + VOCAB * h + VOCAB;
}

static uint32_t pow10u(uint32_t nd) { uint32_t p = 1; while (nd--) p *= 10u; return p; }

void oracle_seq2seq_queries(uint64_t seed, uint32_t generation, uint32_t B, uint32_t nd,
                            int32_t* enc_tokens, int32_t* dec_tokens, int32_t* targets)
{
    const uint32_t range = pow10u(nd), Te = 2 * nd + 1, Td = nd + 1;
    for (uint32_t i = 0; i < B; ++i) {
        uint32_t w[4];
        oracle_stream_words(seed, 6u, generation, 0u, i, w);
        const uint32_t a = (uint32_t)(((uint64_t)w[0] * range) >> 32);
        const uint32_t b = (uint32_t)(((uint64_t)w[1] * range) >> 32);
        const uint32_t sum = a + b;
        int32_t* e = enc_tokens + (size_t)i * Te;
        uint32_t div = range / 10u;
        for (uint32_t k = 0; k < nd; ++k, div /= 10u) {
            e[k] = (int32_t)((a / div) % 10u);
            e[nd + 1 + k] = (int32_t)((b / div) % 10u);
        }
        e[nd] = TOK_PLUS;
        int32_t* t = targets + (size_t)i * Td;
        div = range;                                   /* the sum has nd + 1 digits */
        for (uint32_t k = 0; k < Td; ++k, div /= 10u) t[k] = (int32_t)((sum / div) % 10u);
        int32_t* d = dec_tokens + (size_t)i * Td;
        d[0] = TOK_EQ;
        for (uint32_t k = 1; k < Td; ++k) d[k] = t[k - 1];
    }
}

/* one LSTM step: gates = Wx[:, token] + Wh . h + b; (h, c) updated in place */
static void lstm_step(const float* Wx, const float* Wh, const float* b, uint32_t h, int token,
                      double* hs, double* cs, double* gates, int bf16)
{
    for (uint32_t r = 0; r < 4 * h; ++r) {
        double acc = 0.0;
        for (uint32_t k = 0; k < h; ++k)
            acc += operand((double)Wh[(size_t)r * h + k], bf16) * operand(hs[k], bf16);
        gates[r] = acc + operand((double)Wx[(size_t)r * VOCAB + token], bf16) + operand((double)b[r], bf16);
    }
    for (uint32_t k = 0; k < h; ++k) {
        const double ig = sigmoid(gates[k]);
        const double fg = sigmoid(gates[h + k]);
        const double gg = tanh(gates[2 * h + k]);
        const double og = sigmoid(gates[3 * h + k]);
        cs[k] = fg * cs[k] + ig * gg;
        hs[k] = og * tanh(cs[k]);
    }
}

double oracle_seq2seq_fitness(const float* params, uint32_t h, uint32_t nd, uint32_t B,
                              const int32_t* enc_tokens, const int32_t* dec_tokens,
                              const int32_t* targets, int bf16, double* accuracy,
                              double* logits_out)
{
    const uint32_t Te = 2 * nd + 1, Td = nd + 1;
    const float* eWx = params;
    const float* eWh = eWx + (size_t)4 * h * VOCAB;
    const float* eb  = eWh + (size_t)4 * h * h;
    const float* dWx = eb + 4 * h;
    const float* dWh = dWx + (size_t)4 * h * VOCAB;
    const float* db  = dWh + (size_t)4 * h * h;
    const float* oW  = db + 4 * h;
    const float* ob  = oW + (size_t)VOCAB * h;

    double* hs = (double*)malloc(sizeof(double) * h);
    double* cs = (double*)malloc(sizeof(double) * h);
    double* gates = (double*)malloc(sizeof(double) * 4 * h);
    double loss = 0.0;
    uint64_t right = 0;
    for (uint32_t i = 0; i < B; ++i) {
        memset(hs, 0, sizeof(double) * h);
        memset(cs, 0, sizeof(double) * h);
        for (uint32_t t = 0; t < Te; ++t)
            lstm_step(eWx, eWh, eb, h, enc_tokens[(size_t)i * Te + t], hs, cs, gates, bf16);
        for (uint32_t t = 0; t < Td; ++t) {
            lstm_step(dWx, dWh, db, h, dec_tokens[(size_t)i * Td + t], hs, cs, gates, bf16);
            double logits[VOCAB];
            for (int o = 0; o < VOCAB; ++o) {
                double acc = 0.0;
                for (uint32_t k = 0; k < h; ++k)
                    acc += operand((double)oW[(size_t)o * h + k], bf16) * operand(hs[k], bf16);
                logits[o] = acc + (double)ob[o];
                if (logits_out) logits_out[((size_t)i * Td + t) * VOCAB + o] = logits[o];
            }
            int best = 0;
            double mx = logits[0];
            for (int o = 1; o < VOCAB; ++o) if (logits[o] > mx) { mx = logits[o]; best = o; }
            double se = 0.0;
            for (int o = 0; o < VOCAB; ++o) se += exp(logits[o] - mx);
            const int target = targets[(size_t)i * Td + t];
            loss += (mx + log(se)) - logits[target];
            right += (best == target);
        }
    }
    free(hs); free(cs); free(gates);
    if (accuracy) *accuracy = (double)right / ((double)B * Td);
    return -loss / ((double)B * Td);
}
