/*
 * gru_policy_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain CPU statement of the small recurrent policy that drives the batched
 * env step in the paper's "GRU rollout (~2M parameters)" rows (Table
 * "PufferLib comparisons") and in its time breakdown (Sec. 4: with a fast
 * env the step is model-bound).  The paper prints neither the network nor its
 * sizes beyond "GRU, about 2M parameters"; the reading taken here is
 *
 *     x      = relu(W_e obs + b_e)                       encoder, obs_dim -> H
 *     r      = sigmoid(W_ir x + b_ir + W_hr h + b_hr)    gated recurrent unit
 *     z      = sigmoid(W_iz x + b_iz + W_hz h + b_hz)    (Cho et al. 2014, in
 *     n      = tanh   (W_in x + b_in + r * (W_hn h + b_hn))   the variant that
 *     h'     = (1 - z) * n + z * h                        applies r after the
 *     logits = W_o h' + b_o                               product, as cuDNN /
 *                                                         torch.nn.GRUCell do)
 *
 * with weight rows stored gate-major [r; z; n], each row one output unit.
 *
 * Precision.
 *  - The cell is a dense contraction followed by smooth functions: nothing in
 *    it decides an integer, so it is written in binary64 (exact products of
 *    the binary32 inputs, sums in binary64, libm exp / tanh) and the device
 *    result is compared within a stated tolerance.  Besides h' the cell
 *    returns, per output, the sum of the absolute values of the products that
 *    entered its three pre-activations, which is what an accumulation-error
 *    bound scales with.
 *  - The encoder output is rounded to bfloat16 (it is a tensor-core operand),
 *    so it is written in binary32 with one fixed order: a chain of fused
 *    multiply-adds starting from the bias, inputs ascending.  fmaf is
 *    correctly rounded, so a second implementation can reproduce every bit.
 *  - The head is the definition logits = W_o h' + b_o evaluated plainly in
 *    binary64 (exact products of the binary32 inputs, sums in binary64, bias
 *    last), like the cell.  It also returns, per logit, |b| + sum |h w|, which
 *    is what the rounding error of any binary32 summation order scales with;
 *    a device result is compared within a bound built from it.
 *  - bfloat16 rounding is round-to-nearest-even on the upper 16 bits.
 *
 * One row (env) at a time, plain loops; shares no code with the CUDA path.
 *
 * Pins (tests without a GPU): the cell against torch.nn.GRUCell in binary64
 * on the CPU (a library routine, same definition), closed forms (zero weights,
 * saturated gates keep or replace h), the encoder against binary64 dot
 * products within its rounding bound, the head against numpy's matrix product
 * in binary64, exact small-integer cases and one-hot weights, bfloat16
 * rounding against known bit patterns and ties.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

/* round-to-nearest-even binary32 -> bfloat16, returned as the binary32 value
 * with the low 16 bits cleared.  NaN stays NaN (quiet bit forced). */
float gp_oracle_bf16_round(float v)
{
    uint32_t u;
    memcpy(&u, &v, 4);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu) != 0u) {
        u |= 0x00400000u;
        u &= 0xFFFF0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7FFFu + lsb;
        u &= 0xFFFF0000u;
    }
    float r;
    memcpy(&r, &u, 4);
    return r;
}

/* out[i] = bfloat16 nearest to the binary64 in[i] (ties to even), as a binary32.
 * One rounding: the binary64 is first cut to binary32 toward zero with a sticky
 * last bit (round to odd), which the final rounding to 8 significant bits cannot
 * tell from the exact value. */
void gp_oracle_bf16_round_f64(const double *in, float *out, size_t count)
{
    for (size_t i = 0; i < count; ++i) {
        double d = in[i];
        float f = (float)d;
        if (f == f && f - f == 0.0f && (double)f != d) {   /* finite and inexact */
            if (fabs((double)f) > fabs(d)) f = nextafterf(f, 0.0f);
            uint32_t u;
            memcpy(&u, &f, 4);
            u |= 1u;
            memcpy(&f, &u, 4);
        }
        out[i] = gp_oracle_bf16_round(f);
    }
}

/* x[n][H] = bf16(relu(b_e[c] + sum_i obs[i] * W_e[c][i])), binary32 fma chain, i ascending */
void gp_oracle_encode(const float *obs, int n, int obs_dim, int H, const float *enc_w,
                      const float *enc_b, float *x_out)
{
    for (int m = 0; m < n; ++m) {
        for (int c = 0; c < H; ++c) {
            float acc = enc_b[c];
            for (int i = 0; i < obs_dim; ++i)
                acc = fmaf(obs[(size_t)m * obs_dim + i], enc_w[(size_t)c * obs_dim + i], acc);
            if (!(acc > 0.0f)) acc = 0.0f;
            x_out[(size_t)m * H + c] = gp_oracle_bf16_round(acc);
        }
    }
}

static double dot64(const float *a, const float *b, int K, double *abs_sum)
{
    double s = 0.0, t = 0.0;
    for (int k = 0; k < K; ++k) {
        double p = (double)a[k] * (double)b[k];
        s += p;
        t += fabs(p);
    }
    *abs_sum += t;
    return s;
}

static double sigmoid64(double v) { return 1.0 / (1.0 + exp(-v)); }

/* h_out[n][H] (binary64, not rounded); abs_sum[n][H] may be NULL. */
void gp_oracle_cell(const float *x, const float *h, int n, int H, const float *w_ih,
                    const float *w_hh, const float *b_ih, const float *b_hh, double *h_out,
                    double *abs_sum)
{
    for (int m = 0; m < n; ++m) {
        const float *xm = x + (size_t)m * H;
        const float *hm = h + (size_t)m * H;
        for (int j = 0; j < H; ++j) {
            double t = 0.0;
            double xr = dot64(xm, w_ih + (size_t)(0 * H + j) * H, H, &t);
            double xz = dot64(xm, w_ih + (size_t)(1 * H + j) * H, H, &t);
            double xn = dot64(xm, w_ih + (size_t)(2 * H + j) * H, H, &t);
            double hr = dot64(hm, w_hh + (size_t)(0 * H + j) * H, H, &t);
            double hz = dot64(hm, w_hh + (size_t)(1 * H + j) * H, H, &t);
            double hn = dot64(hm, w_hh + (size_t)(2 * H + j) * H, H, &t);
            double r = sigmoid64(xr + (double)b_ih[0 * H + j] + hr + (double)b_hh[0 * H + j]);
            double z = sigmoid64(xz + (double)b_ih[1 * H + j] + hz + (double)b_hh[1 * H + j]);
            double c = tanh(xn + (double)b_ih[2 * H + j] + r * (hn + (double)b_hh[2 * H + j]));
            h_out[(size_t)m * H + j] = (1.0 - z) * c + z * (double)hm[j];
            if (abs_sum) abs_sum[(size_t)m * H + j] = t;
        }
    }
}

/* logits[n][A] = b_o[a] + sum_k h[k] * W_o[a][k] in binary64; abs_sum[n][A]
 * (may be NULL) = |b_o[a]| + sum_k |h[k] * W_o[a][k]|. */
void gp_oracle_head(const float *h, int n, int H, int A, const float *head_w, const float *head_b,
                    double *logits, double *abs_sum)
{
    for (int m = 0; m < n; ++m) {
        for (int a = 0; a < A; ++a) {
            double t = 0.0;
            double s = dot64(h + (size_t)m * H, head_w + (size_t)a * H, H, &t);
            logits[(size_t)m * A + a] = s + (double)head_b[a];
            if (abs_sum) abs_sum[(size_t)m * A + a] = t + fabs((double)head_b[a]);
        }
    }
}
