/*
 * gru_policy.h -- C ABI of the B200 recurrent-policy library: the small GRU
 * network that produces the actions of a batched environment step when the
 * policy runs in the loop.
 *
 * This is the setting of the paper's "GRU rollout (~2M parameters)" rows (Table
 * "PufferLib comparisons") and of its time breakdown (Sec. 4: once the env is
 * fast, the step is bound by the model).  The paper gives the network only as
 * "GRU, about 2M parameters"; the network here is
 *
 *     x      = relu(W_e obs + b_e)                          encoder, obs_dim -> H
 *     r      = sigmoid(W_ir x + b_ir + W_hr h + b_hr)
 *     z      = sigmoid(W_iz x + b_iz + W_hz h + b_hz)
 *     n      = tanh   (W_in x + b_in + r * (W_hn h + b_hn))
 *     h'     = (1 - z) * n + z * h
 *     logits = W_o h' + b_o                                 head, H -> n_actions
 *
 * (the gated recurrent unit of Cho et al. 2014 in the variant that applies the
 * reset gate after the hidden-side product).  H = 576 with obs_dim 6 and 3
 * actions has 2.0 M parameters.
 *
 * Arithmetic.
 *  - gru_policy_encode: binary32, one fused multiply-add per input starting from
 *    the bias, inputs in ascending order; rectifier; the result is rounded to
 *    bfloat16 (round to nearest even).  Reproducible bit for bit.
 *  - gru_policy_cell: the six matrix products run on the tensor cores with
 *    bfloat16 operands (x, h and the weights, which gru_policy_create rounds to
 *    bfloat16 once) and binary32 accumulation; biases, gates and the blend are
 *    binary32; h' is rounded to bfloat16.  The accumulation order inside the
 *    tensor cores is not specified, so h' is defined up to that: it agrees with
 *    an exact evaluation to within one bfloat16 rounding plus a binary32
 *    accumulation error (see the parity tests for the bound).
 *  - gru_policy_head: the definition logits = W_o h' + b_o, summed in binary32 in
 *    this library's own order: the hidden units are taken in blocks of 32 (the
 *    cell kernel's epilogue tile); a block's partial sum is a chain of fused
 *    multiply-adds from zero over its units in ascending order; the logit is the
 *    bias plus the partial sums added one by one in block order.  The result is
 *    within (H + H/32 + 1) * 2^-24 * (|b| + sum |h w|) of the exact value (one
 *    rounding per fused multiply-add, per partial sum added and for the bias), and
 *    the same bits on every call.  gru_policy_cell_head forms the partial sums in
 *    the cell's epilogue, where each block of h' is produced, and gives the bits of
 *    gru_policy_head applied to its h'.
 *
 * Conventions.  Parameters are given to gru_policy_create as HOST float arrays,
 * rows = output units, gate blocks of w_ih / w_hh / b_ih / b_hh in the order
 * r, z, n; the library keeps its own device copies.  Every other pointer is a
 * DEVICE pointer owned by the caller; x and h buffers hold bfloat16 [n][H],
 * row-major, 16-byte aligned.  Calls enqueue on the handle's stream and return
 * (gru_policy_status synchronises).  The library allocates only in
 * gru_policy_create.  Return 0 or a negative GRU_POLICY_E* code; no exceptions,
 * aborts, traps or printing; no CPU fallback.
 */
#ifndef GRU_POLICY_H_
#define GRU_POLICY_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GRU_POLICY_OK        0
#define GRU_POLICY_EINVAL   (-1)  /* bad size (hidden not a multiple of 64, n < 1, ...) */
#define GRU_POLICY_ENULL    (-2)  /* required pointer is NULL */
#define GRU_POLICY_EALIGN   (-3)  /* x / h pointer not 16-byte aligned, obs not 8-byte aligned */
#define GRU_POLICY_ECUDA    (-4)  /* a CUDA runtime call or launch failed */
#define GRU_POLICY_ENOMEM   (-5)  /* allocation failed */
#define GRU_POLICY_ETIMEOUT (-6)  /* a kernel gave up a bounded wait; its output is invalid */

#define GRU_POLICY_MAX_HIDDEN 1024
#define GRU_POLICY_MAX_OBS    16
#define GRU_POLICY_MAX_ACTIONS 8

typedef struct gru_policy gru_policy;

/* hidden: multiple of 64, 64..GRU_POLICY_MAX_HIDDEN.  All eight arrays are host
 * float32: enc_w[hidden][obs_dim], enc_b[hidden], w_ih[3*hidden][hidden],
 * w_hh[3*hidden][hidden], b_ih[3*hidden], b_hh[3*hidden],
 * head_w[n_actions][hidden], head_b[n_actions].  w_ih and w_hh are rounded to
 * bfloat16; the rest stays binary32. */
int gru_policy_create(gru_policy **out, int hidden, int obs_dim, int n_actions,
                      const float *enc_w, const float *enc_b, const float *w_ih, const float *w_hh,
                      const float *b_ih, const float *b_hh, const float *head_w,
                      const float *head_b);
int gru_policy_destroy(gru_policy *p);
int gru_policy_set_stream(gru_policy *p, void *cuda_stream);

/* x_out[n][H] (bfloat16) = encoder(obs[n][obs_dim] float32, 8-byte aligned).  If done is not
 * NULL (uint8[n]) and h is not NULL, row m of h (bfloat16 [n][H]) is set to zero
 * where done[m] != 0: a finished episode starts the next one from a zero state. */
int gru_policy_encode(gru_policy *p, const float *obs, const uint8_t *done, void *h, void *x_out,
                      int n);

/* h_out[n][H] = cell(x[n][H], h_in[n][H]), all bfloat16.  h_out must not overlap
 * x or h_in. */
int gru_policy_cell(gru_policy *p, const void *x, const void *h_in, void *h_out, int n);

/* logits[n][n_actions] (float32) = head(h[n][H] bfloat16). */
int gru_policy_head(gru_policy *p, const void *h, float *logits, int n);

/* Bytes of device scratch gru_policy_cell_head needs for n envs (0 if p is NULL or n < 1). */
size_t gru_policy_workspace_bytes(const gru_policy *p, int n);

/* gru_policy_cell followed by gru_policy_head on its result, with the head's partial
 * sums formed inside the cell kernel: h_out as gru_policy_cell, logits as
 * gru_policy_head(h_out).  workspace: device scratch of gru_policy_workspace_bytes(p, n)
 * bytes, 16-byte aligned, owned by the caller.  Needs n_actions <= 4 and hidden <= 896
 * (GRU_POLICY_EINVAL otherwise: call the two entry points separately). */
int gru_policy_cell_head(gru_policy *p, const void *x, const void *h_in, void *h_out, float *logits,
                         void *workspace, int n);

/* Synchronises the stream; GRU_POLICY_ETIMEOUT if any kernel since the last call
 * gave up a wait (clears the flag), GRU_POLICY_ECUDA on a CUDA error, else 0. */
int gru_policy_status(gru_policy *p);

int gru_policy_hidden(const gru_policy *p);
/* kernels launched through this handle so far */
int64_t gru_policy_launch_count(const gru_policy *p);
const char *gru_policy_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* GRU_POLICY_H_ */
