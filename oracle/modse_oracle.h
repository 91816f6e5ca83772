/*
 * MoDSE layer oracle: plain fp64 CPU code, loops only.
 *
 * TEST INFRASTRUCTURE ONLY.  This is the slow, by-eye-checkable definition of
 * what the Mixture-of-Diverse-Size-Experts feed-forward layer computes.  It is
 * used by the test-suite, by the smoke check and by the benchmark's CPU
 * baseline leg; the CUDA library never includes, links or calls it, and it
 * shares no code with the CUDA sources.
 *
 * Notation (follows the paper): T tokens, d = model width (input size), N
 * experts, k = top-k, h[e] = hidden width of diverse-size expert e ("h-hat_i",
 * Sec. 3.1), S = sum_e h[e], off[e] = sum_{e'<e} h[e'].
 *
 * Layouts (all row-major, all double):
 *   x        [T, d]
 *   w_router [N, d]            one logit row per expert (W_g of Eq. 2's H(x))
 *   w_gate   [S, d]            expert e owns rows off[e] .. off[e]+h[e]-1
 *   w_up     [S, d]            same
 *   w_down   expert e is a [d, h[e]] block at element offset d*off[e]
 *
 * Parity pins (tests/test_oracle_*.py): routing invariants and brute-force
 * sort; closed form g0 = sigmoid(z0-z1); dense-mask evaluation of Eq. 1;
 * one-expert top-1 == dense SwiGLU FFN via library matmul/silu; equal-width
 * experts == standard top-2 MoE; central finite differences for every
 * gradient; softmax-Jacobian identities.  The paper prints no worked numerical
 * example of a layer output, so absolute values are pinned by those only.
 *
 * Return value of every function: 0 on success, -1 bad argument, -2 a
 * non-finite router logit was met (out of contract), -3 out of memory.
 */
#ifndef MODSE_ORACLE_H
#define MODSE_ORACLE_H
#ifdef __cplusplus
extern "C" {
#endif

/* Eq. 2-3 with H(x) = x . W_g : logits, top-k (ties -> lower expert index),
 * softmax over the kept logits, then per-expert counts, exclusive offsets and
 * the stable permutation (rows of an expert in ascending token order; expert
 * groups in ascending expert order).
 *   z           [T,N] out, may be NULL
 *   topk_idx    [T,k] out, slot 0 = largest logit
 *   topk_gate   [T,k] out
 *   counts      [N]   out      counts_slot [k,N] out (per pick slot, as the
 *                              paper's Appendix A tables log them)
 *   offsets     [N+1] out
 *   row_of      [T,k] out      token_of [k*T] out (inverse map)          */
int modse_oracle_route(int T, int d, int N, int k,
                       const double *x, const double *w_router,
                       double *z, int *topk_idx, double *topk_gate,
                       int *counts, int *counts_slot, int *offsets,
                       int *row_of, int *token_of);

/* Eq. 4 for the listed tokens: y_t = sum_j g[t,j] * E_{idx[t,j]}(x_t), each
 * expert a bias-free SwiGLU FFN  E(x) = W_down (silu(W_gate x) * (W_up x)).
 *   sel   [n_sel] token indices (NULL = tokens 0..n_sel-1)
 *   y_sel [n_sel,d] out;  o_sel [n_sel,k,d] out or NULL (ungated expert outputs) */
int modse_oracle_forward_tokens(int T, int d, int N, int k, const int *h,
                                const double *x, const double *w_gate,
                                const double *w_up, const double *w_down,
                                const int *topk_idx, const double *topk_gate,
                                int n_sel, const int *sel,
                                double *y_sel, double *o_sel);

/* Exact gradient of the forward with the top-k selection held fixed, for the
 * listed tokens only: dx (expert path + router path), dg = <dY_t, o_(t,j)> and
 * dz (Jacobian of the softmax over the kept logits).
 *   dx_sel [n_sel,d], dg_sel [n_sel,k], dz_sel [n_sel,N]; any may be NULL   */
int modse_oracle_backward_tokens(int T, int d, int N, int k, const int *h,
                                 const double *x, const double *w_router,
                                 const double *w_gate, const double *w_up,
                                 const double *w_down, const int *topk_idx,
                                 const double *topk_gate, const double *dy,
                                 int n_sel, const int *sel,
                                 double *dx_sel, double *dg_sel, double *dz_sel);

/* Weight-gradient rows for the listed (expert, hidden unit) pairs, summed over
 * every token routed to that expert:
 *   dwg_rows [n_rows,d]  row r of dW_gate_e      dwu_rows likewise for W_up
 *   dwd_cols [n_rows,d]  column r of dW_down_e (all d output rows)          */
int modse_oracle_wgrad_rows(int T, int d, int N, int k, const int *h,
                            const double *x, const double *w_gate,
                            const double *w_up, const double *w_down,
                            const int *topk_idx, const double *topk_gate,
                            const double *dy, int n_rows, const int *rows_e,
                            const int *rows_r, double *dwg_rows,
                            double *dwu_rows, double *dwd_cols);

/* Whole backward, every output (sized like the matching input); dg [T,k] and
 * dz [T,N] may be NULL.  Empty experts get zero weight gradients.          */
int modse_oracle_backward(int T, int d, int N, int k, const int *h,
                          const double *x, const double *w_router,
                          const double *w_gate, const double *w_up,
                          const double *w_down, const int *topk_idx,
                          const double *topk_gate, const double *dy,
                          double *dx, double *dw_router, double *dw_gate,
                          double *dw_up, double *dw_down, double *dg, double *dz);

/* Switch-style auxiliary load-balance loss of Eq. 7-10:
 *   L_a = alpha * N * sum_i f_i * P_i,  f_i = share of tokens whose arg-max
 *   probability is expert i,  P_i = mean full-softmax probability of expert i.
 *   f [N], P [N] out (may be NULL); dz_aux [T,N] out or NULL = dL_a/dz with f
 *   held constant (it is piecewise constant in z).                         */
int modse_oracle_aux_loss(int T, int N, const double *z, double alpha,
                          double *loss, double *f, double *P, double *dz_aux);

/* Second term of H(x) (Sec. 2, Eq. 2 with Eq. 4-5): r[t,i] = RMSNorm(Softplus(x W_n))_i with the
 * RMS taken over the N expert entries of token t and a scalar gamma; u_out [T,N] (may be NULL)
 * receives x W_n.                                                                            */
int modse_oracle_noise_term(int T, int d, int N, const double *x, const double *w_noise,
                            double gamma, double eps, double *r, double *u_out);

/* Its gradient for dz = dL/dH [T,N]: dx_add [T,d] (to be added to dx), dw_noise [N,d], dgamma. */
int modse_oracle_noise_backward(int T, int d, int N, const double *x, const double *w_noise,
                                double gamma, double eps, const double *dz,
                                double *dx_add, double *dw_noise, double *dgamma);

/* Top-k, gates and permutation tables from given logits z [T,N] (same rules as modse_oracle_route). */
int modse_oracle_route_from_logits(int T, int N, int k, const double *z, int *topk_idx,
                                   double *topk_gate, int *counts, int *counts_slot, int *offsets,
                                   int *row_of, int *token_of);

int modse_oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
