/*
 * Sequential fp64 CPU oracle for the seven credit-assignment recurrences.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain definition of what the
 * CUDA library must compute: one row at a time, one timestep at a time, in
 * double precision, written from the boundary *semantics* of the paper
 * (Section 3.2) as branches -- not from (alpha, beta) pairs -- so that it
 * shares neither code nor structure with the GPU scan.  Only the tests, the
 * smoke check and the benchmark's cpu_baseline / reference legs may call it.
 *
 * Conventions (all row-major, element (n,t) at n*T+t):
 *   - fp32 inputs are widened element by element; outputs are fp64.
 *   - masks are uint8, non-zero = true.  `term` is d^term, `trunc` is d^trunc
 *     (NULL = all false); d_t = term_t OR trunc_t is the flag that severs the
 *     recurrence (Table 1 caption).
 *   - `bv` is the 2-D per-step truncation continuation value
 *     bootstrap_values[n,t] (Section 3.2 "Truncated steps"); read only where
 *     trunc_t is set and term_t is not.
 *   - `boot` is the 1-D window-edge value for s_T (NULL = 0, the
 *     HAS_BOOTSTRAP=False case of Section 4.2).
 *
 * Successor value of step t (Section 3.2), used by every backward routine:
 *     0          if term_t                      (episode ended: zero successor)
 *     bv[t]      else if trunc_t                (supplied continuation value)
 *     boot       else if t == T-1               (rollout-window edge)
 *     X[t+1]     otherwise
 * "term wins" when both flags are set: the paper keeps the (1 - d^term_t)
 * factor on the successor value in every row of Table 1.
 *
 * The recurrence continues from t into t+1 only when neither flag is set and
 * t+1 is inside the buffer.
 *
 * Every function below is pinned by tests that do not use this file's
 * formulas: Table 1's literal (alpha, beta, carry) solved by the explicit
 * O(T^2) sum, closed forms, special cases (gamma=0, lambda=0, lambda=1),
 * cross-algorithm identities and the paper's 4-step expansion.  The routines
 * beyond the seven (Retrace from [N,T,A] tensors, vector traces with a shared
 * or a per-component decay, GAE with observation-skip masking) are pinned by
 * reduction to the seven (gather / compaction / per-component equality) and by
 * the unrolled sum of Eq. 1.  Nothing here is "parity unpinned".
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>

static inline int flag(const uint8_t* m, int64_t i) { return m != NULL && m[i] != 0; }

/* Successor value per Section 3.2; `next` is the in-buffer X[t+1] (ignored
 * at flagged steps and at t == T-1). */
static inline double successor(int term, int trunc, int last, double bv_t, double boot, double next) {
    if (term) return 0.0;
    if (trunc) return bv_t;
    if (last) return boot;
    return next;
}

/* GAE (Section 3.3.1): A_t = delta_t + gamma*lambda*A_{t+1} inside an
 * episode, A_T = 0; delta_t = r_t + gamma*V(s_{t+1}) - V(s_t) with the
 * successor value of Section 3.2.  ret = A + V (optional). */
void rlcs_oracle_gae(const float* r, const float* V, const uint8_t* term, const uint8_t* trunc,
                     const float* bv, const float* boot, double* adv, double* ret,
                     int64_t N, int64_t T, double gamma, double lambda) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double A_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const double vn = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b,
                                        last ? 0.0 : (double)V[o + t + 1]);
            const double delta = (double)r[o + t] + gamma * vn - (double)V[o + t];
            const int cont = !tm && !tr && !last;
            const double A = cont ? delta + gamma * lambda * A_next : delta;
            adv[o + t] = A;
            if (ret) ret[o + t] = A + (double)V[o + t];
            A_next = A;
        }
    }
}

/* GAE with observation-skip masking (planned in Section 9.2: the recurrence is carried across masked
 * tokens with beta_t = 1).  Reading taken here: a masked step is transparent -- it adds no TD
 * error and no discount, A_t = A_{t+1}, and the value that earlier steps see through it is the
 * value of the next unmasked step, W_t = W_{t+1}; an unmasked step is the GAE step of Section 3.3.1
 * with successor value W_{t+1}.  Termination and truncation flags sever the recurrence as in Section
 * 3.2 wherever they stand: at a flagged masked step A_t = 0 and W_t is the flag's successor value.
 * Outputs: adv = A, ret = A + W (optional), filled = W (optional).  Without flags on masked steps the
 * result at the unmasked steps is plain GAE of the sequence with the masked steps deleted. */
void rlcs_oracle_gae_skip(const float* r, const float* V, const uint8_t* term, const uint8_t* trunc,
                          const float* bv, const float* boot, const uint8_t* skip, double* adv, double* ret,
                          double* filled, int64_t N, int64_t T, double gamma, double lambda) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double A_next = 0.0, W_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const double vn = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b, W_next);
            const int cont = !tm && !tr && !last;
            double A, W;
            if (flag(skip, o + t)) {
                A = cont ? A_next : 0.0;
                W = vn;                                   /* cont: the next unmasked value, passed through */
            } else {
                const double delta = (double)r[o + t] + gamma * vn - (double)V[o + t];
                A = cont ? delta + gamma * lambda * A_next : delta;
                W = (double)V[o + t];
            }
            adv[o + t] = A;
            if (ret) ret[o + t] = A + W;
            if (filled) filled[o + t] = W;
            A_next = A;
            W_next = W;
        }
    }
}

/* TD(lambda) returns (Section 3.3.4):
 * G_t = r_t + gamma*[(1-lambda)*V(s_{t+1}) + lambda*G_{t+1}].  Where the
 * recurrence is severed (flag or window edge) the continuation G_{t+1} is the
 * successor value itself, so G_t = r_t + gamma*successor -- the paper's
 * window-edge identity G_{T-1} = r_{T-1} + gamma*V(s_T) and its interior
 * truncation rule alpha_t = r_t + gamma*V(s^true_{t+1}). */
void rlcs_oracle_td_lambda(const float* r, const float* V, const uint8_t* term, const uint8_t* trunc,
                           const float* bv, const float* boot, double* G,
                           int64_t N, int64_t T, double gamma, double lambda) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double G_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const double x = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b,
                                       last ? 0.0 : (double)V[o + t + 1]);
            const int cont = !tm && !tr && !last;
            const double gn = cont ? G_next : x;
            const double g = (double)r[o + t] + gamma * ((1.0 - lambda) * x + lambda * gn);
            G[o + t] = g;
            G_next = g;
        }
    }
}

/* Discounted returns (Section 3.3.4, the lambda=1 case with no value
 * function): G_t = r_t + gamma*G_{t+1}; at a severed step the continuation is
 * 0 (terminated), bv[t] (truncated) or boot (window edge). */
void rlcs_oracle_discounted_return(const float* r, const uint8_t* term, const uint8_t* trunc,
                                   const float* bv, const float* boot, double* G,
                                   int64_t N, int64_t T, double gamma) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double G_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const int cont = !tm && !tr && !last;
            const double gn = cont ? G_next
                                   : successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b, 0.0);
            const double g = (double)r[o + t] + gamma * gn;
            G[o + t] = g;
            G_next = g;
        }
    }
}

/* V-Trace (Section 3.3.2).  rho_t = min(rho_bar, e^{lr_t}), c_t = min(c_bar,
 * e^{lr_t}); Delta_t = rho_t*(r_t + gamma*V(s_{t+1}) - V(s_t)) +
 * gamma*c_t*Delta_{t+1}, Delta_T = 0; v_t = V(s_t) + Delta_t; then
 * A_t = rho_t*(r_t + gamma*v_{t+1} - V(s_t)), where v_{t+1} at a severed step
 * is the successor value (0 / bv / boot), as when the bootstrap value is
 * appended to the targets. */
void rlcs_oracle_vtrace(const float* r, const float* V, const float* log_rho, const uint8_t* term,
                        const uint8_t* trunc, const float* bv, const float* boot, double* vs,
                        double* pg_adv, int64_t N, int64_t T, double gamma, double rho_bar,
                        double c_bar) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double D_next = 0.0, vs_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const double raw = exp((double)log_rho[o + t]);
            const double rho = raw < rho_bar ? raw : rho_bar;
            const double c = raw < c_bar ? raw : c_bar;
            const double x = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b,
                                       last ? 0.0 : (double)V[o + t + 1]);
            const int cont = !tm && !tr && !last;
            const double delta = rho * ((double)r[o + t] + gamma * x - (double)V[o + t]);
            const double D = cont ? delta + gamma * c * D_next : delta;
            const double v = (double)V[o + t] + D;
            const double vn = cont ? vs_next : x;
            vs[o + t] = v;
            if (pg_adv) pg_adv[o + t] = rho * ((double)r[o + t] + gamma * vn - (double)V[o + t]);
            D_next = D;
            vs_next = v;
        }
    }
}

/* Retrace(lambda) (Section 3.3.3).  c_t = lambda*min(c_bar, e^{lr_t});
 * Delta_t = r_t + gamma*E_pi Q(s_{t+1},.) - Q(s_t,a_t) +
 * gamma*c_{t+1}*Delta_{t+1}, Delta_T = 0 -- the decay that multiplies
 * Delta_{t+1} is the NEXT step's trace coefficient (index shift).  eq[n,t] is
 * E_pi Q(s_t,.), so the successor value of step t reads eq[n,t+1]; boot is
 * E_pi Q(s_T,.).  Output: Q(s_t,a_t) + Delta_t. */
void rlcs_oracle_retrace(const float* r, const float* q, const float* eq, const float* log_rho,
                         const uint8_t* term, const uint8_t* trunc, const float* bv,
                         const float* boot, double* target, int64_t N, int64_t T, double gamma,
                         double lambda, double c_bar) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double D_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            const double x = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b,
                                       last ? 0.0 : (double)eq[o + t + 1]);
            const int cont = !tm && !tr && !last;
            double D = (double)r[o + t] + gamma * x - (double)q[o + t];
            if (cont) {
                const double raw = exp((double)log_rho[o + t + 1]);
                const double c_next = lambda * (raw < c_bar ? raw : c_bar);
                D += gamma * c_next * D_next;
            }
            target[o + t] = (double)q[o + t] + D;
            D_next = D;
        }
    }
}

/* Retrace(lambda) from [N,T,A] tensors (Section 3.3.3 with the input form of Section 7.3): per step
 * Q(s_t,a_t) = Q[n,t,a_t], E_pi Q(s_t,.) = sum_a pi[n,t,a] Q[n,t,a], and the importance ratio
 * pi[n,t,a_t] / mu[n,t,a_t]; then the same recurrence as rlcs_oracle_retrace, with the decay built
 * from the NEXT step's ratio: c_{t+1} = lambda * min(c_bar, ratio_{t+1}). */
void rlcs_oracle_retrace_probs(const float* r, const float* Q, const float* pi, const float* mu, const int32_t* act,
                               const uint8_t* term, const uint8_t* trunc, const float* bv, const float* boot,
                               double* target, int64_t N, int64_t T, int64_t A, double gamma, double lambda,
                               double c_bar) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        const double b = boot ? (double)boot[n] : 0.0;
        double D_next = 0.0;
        for (int64_t t = T - 1; t >= 0; --t) {
            const int tm = flag(term, o + t), tr = flag(trunc, o + t), last = (t == T - 1);
            double eq_next = 0.0;                       /* E_pi Q(s_{t+1}, .) */
            if (!last)
                for (int64_t a = 0; a < A; ++a) eq_next += (double)pi[(o + t + 1) * A + a] * (double)Q[(o + t + 1) * A + a];
            const double x = successor(tm, tr, last, (tr && !tm) ? (double)bv[o + t] : 0.0, b, eq_next);
            const int cont = !tm && !tr && !last;
            const double q_sa = (double)Q[(o + t) * A + act[o + t]];
            double D = (double)r[o + t] + gamma * x - q_sa;
            if (cont) {
                const int64_t an = act[o + t + 1];
                const double raw = (double)pi[(o + t + 1) * A + an] / (double)mu[(o + t + 1) * A + an];
                D += gamma * lambda * (raw < c_bar ? raw : c_bar) * D_next;
            }
            target[o + t] = q_sa + D;
            D_next = D;
        }
    }
}

/* Eligibility trace, scalar form (Section 3.3.5), forward in time:
 * z_t = gamma*lambda*(1 - d_{t-1})*z_{t-1} + x_t, d_{-1} := 0, z_{-1} = 0.
 * `d` is the combined flag (term OR trunc), as the forward scans take it. */
void rlcs_oracle_elig_trace(const float* x, const uint8_t* d, double* z, int64_t N, int64_t T,
                            double gamma, double lambda) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        double z_prev = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            const int carry = (t > 0) && !flag(d, o + t - 1);
            const double zt = carry ? (double)x[o + t] + gamma * lambda * z_prev : (double)x[o + t];
            z[o + t] = zt;
            z_prev = zt;
        }
    }
}

/* Vector-valued eligibility trace (Table 1, vector form): x, z are [N,T,D]; one scalar decay per step. */
void rlcs_oracle_elig_trace_vec(const float* x, const uint8_t* d, double* z, int64_t N, int64_t T, int64_t D,
                                double gamma, double lambda) {
    for (int64_t n = 0; n < N; ++n)
        for (int64_t t = 0; t < T; ++t) {
            const int carry = (t > 0) && !flag(d, n * T + t - 1);
            for (int64_t c = 0; c < D; ++c) {
                const int64_t i = (n * T + t) * D + c;
                z[i] = carry ? (double)x[i] + gamma * lambda * z[i - D] : (double)x[i];
            }
        }
}

/* Eligibility trace with a decay per component and step (per-dimension beta_t, Section 9.1): Eq. 1
 * component by component, z_t[c] = x_t[c] + beta_t[c] * z_{t-1}[c], the carry severed after a flag. */
void rlcs_oracle_elig_trace_vec_beta(const float* x, const float* beta, const uint8_t* d, double* z, int64_t N, int64_t T,
                                     int64_t D) {
    for (int64_t n = 0; n < N; ++n)
        for (int64_t t = 0; t < T; ++t) {
            const int carry = (t > 0) && !flag(d, n * T + t - 1);
            for (int64_t c = 0; c < D; ++c) {
                const int64_t i = (n * T + t) * D + c;
                z[i] = carry ? (double)x[i] + (double)beta[i] * z[i - D] : (double)x[i];
            }
        }
}

/* Episodic prefix sum (Section 3.3.6), forward in time.  ends_at (default):
 * C_t = x_t + (1 - d_{t-1})*C_{t-1}; starts_at: C_t = x_t + (1 - d_t)*C_{t-1}.
 * C_{-1} = 0 in both, so C_0 = x_0 whatever d_0 is. */
void rlcs_oracle_episodic_prefix_sum(const float* x, const uint8_t* d, double* C, int64_t N,
                                     int64_t T, int starts_at) {
    for (int64_t n = 0; n < N; ++n) {
        const int64_t o = n * T;
        double c_prev = 0.0;
        for (int64_t t = 0; t < T; ++t) {
            const int reset = (t == 0) || (starts_at ? flag(d, o + t) : flag(d, o + t - 1));
            const double ct = reset ? (double)x[o + t] : (double)x[o + t] + c_prev;
            C[o + t] = ct;
            c_prev = ct;
        }
    }
}

/* Generic first-order linear recurrence on precomputed fp64 coefficients
 * (Eq. 1), one row: backward A_t = alpha_t + beta_t*A_{t+1} with A_T = carry,
 * or the forward mirror A_t = alpha_t + beta_t*A_{t-1} with A_{-1} = carry. */
void rlcs_oracle_linear_recurrence(const double* alpha, const double* beta, double carry,
                                   double* A, int64_t T, int forward) {
    double prev = carry;
    if (forward) {
        for (int64_t t = 0; t < T; ++t) { prev = alpha[t] + beta[t] * prev; A[t] = prev; }
    } else {
        for (int64_t t = T - 1; t >= 0; --t) { prev = alpha[t] + beta[t] * prev; A[t] = prev; }
    }
}

/* The affine-pair combine of Eq. 2: (aB,bB) (+) (aA,bA) = (aB + bB*aA, bA*bB),
 * B the chronologically earlier operand for backward scans. */
void rlcs_oracle_combine(double aB, double bB, double aA, double bA, double* a_out, double* b_out) {
    *a_out = aB + bB * aA;
    *b_out = bA * bB;
}
