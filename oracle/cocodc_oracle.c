/*
 * CPU oracle for CoCoDC's per-fragment outer synchronisation step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, element-by-element
 * restatement of the paper's equations in double precision, evaluated on the
 * exact fp32 input bits.  Nothing in the product may call it: it exists so
 * that tests (and the benchmark's CPU-baseline leg) have an independent answer
 * to compare the CUDA library with.  It shares no code with that library.
 *
 * Notation follows the paper (Section 2.1, Section 3.1):
 *   b   = theta^m_{p,t_p}   worker m's fragment when the sync was initiated
 *   a   = theta^m_{p,t_l}   the same fragment now, tau local steps later
 *   thg = theta^g_{p,t_p-H} global state of the fragment from its last sync
 *   u   = outer-optimizer momentum buffer (kept in the direction of Delta)
 *   G   = theta^g_{p,t_p}   new global state after the outer update
 *
 * Readings taken where the paper is silent or inconsistent (listed with their
 * reasons in the design notes of the repository):
 *   - outer optimizer = SGD with Nesterov momentum, no dampening, no weight
 *     decay, fed the gradient -Delta:  u' = mu*u + Delta ; G = thg + eta*(Delta + mu*u')
 *   - the "outer product" symbol of Eq. 6 acts element-wise
 *   - Delta theta^m_{p,t_p} of Eq. 6 is G - b, as the chain of Eq. 5 defines it
 *   - the divisor H of Eq. 6 is the number of local steps
 *   - sign modes: 0 FORWARD  g = (a-b)/tau, Eq. 7 as printed
 *                 1 PRINTED  g = (b-a)/tau (Eq. 4 as printed), Eq. 7 as printed
 *                 2 DESCENT  g = (b-a)/tau, Eq. 7 with its sign flipped
 *   - tau = 0 means no overlap: the target is G itself (Eq. 4 is not evaluated)
 */

#include <math.h>
#include <stddef.h>

enum { COMP_NONE = 0, COMP_TAYLOR = 1 };
enum { SIGN_FORWARD = 0, SIGN_PRINTED = 1, SIGN_DESCENT = 2 };

/* Section 3.1, Eq. 4-7 (Algorithm 1) for one element of one worker, followed
 * by the blend of Eq. 3 with mixing factor alpha (alpha = 1 is Eq. 7's
 * assignment). */
static double merged_value(double a, double b, double G, double lambda, double alpha,
                           long tau, long H, int comp_mode, int sign_mode)
{
    double target;
    if (comp_mode == COMP_NONE || tau == 0) {
        target = G;                                            /* Eq. 3 blends G itself */
    } else {
        double sgn4 = (sign_mode == SIGN_FORWARD) ? 1.0 : -1.0;
        double sgn7 = (sign_mode == SIGN_DESCENT) ? -1.0 : 1.0;
        double g = sgn4 * (a - b) / (double)tau;               /* Eq. 4: local change rate   */
        double D = G - b;                                      /* Eq. 5: theta^g_tp - theta^m_tp */
        double gcorr = g + lambda * g * g * (D / (double)H);   /* Eq. 6                       */
        target = G + sgn7 * gcorr * (double)tau;               /* Eq. 7                       */
    }
    return (1.0 - alpha) * a + alpha * target;                 /* Eq. 3                       */
}

/*
 * One pass of the outer step over n consecutive elements of a fragment.
 *
 *   snap[m*snap_stride + i]  = b for worker m, element i
 *   now [m*now_stride  + i]  = a for worker m, element i
 *   theta_g[i], u[i]         = thg, momentum
 *
 * Outputs (double): theta_g_out[i] = G, u_out[i] = u', delta_out[i] = Delta,
 * now_out[m*n + i] = merged local value.  do_merge = 0 leaves now_out alone.
 * Returns sum_i Delta_i^2 accumulated in element order (for Eq. 10's norm).
 *
 * Worker-per-device deployment (Section 2.1: each worker all-reduces its pseudo-gradient): if
 * n_recv > 0, recv_sums[0..n_recv-1] hold, per element, sums of pseudo-gradients (fp32) that together
 * cover ALL M_total workers - one buffer if the exchange has already added them up, one per contributing
 * device otherwise - and Eq. 1's mean is their total / M_total; the M local workers in snap/now are then
 * only merged.  n_recv == 0: the mean is formed from the M stacked workers as above.
 */
double cocodc_oracle_outer_elements(
    long n, int M,
    const float *snap, long snap_stride,
    const float *now, long now_stride,
    const float *theta_g, const float *u,
    double eta, double mu, double lambda, double alpha, long tau, long H,
    int comp_mode, int sign_mode, int do_merge,
    const float *const *recv_sums, int n_recv, int M_total,
    double *now_out, double *theta_g_out, double *u_out, double *delta_out)
{
    long double sumsq = 0.0L;
    for (long i = 0; i < n; ++i) {
        double thg = (double)theta_g[i];
        double Delta;
        if (n_recv > 0) {
            double total = 0.0;                                  /* Eq. 1 from the exchanged sums */
            for (int r = 0; r < n_recv; ++r)
                total += (double)recv_sums[r][i];
            Delta = total / (double)M_total;
        } else {
            /* pseudo-gradient of every worker (Section 2.1) and their mean, Eq. 1:
             * differences first, summed in worker order, then divided by M */
            double sum = 0.0;
            for (int m = 0; m < M; ++m) {
                double delta_m = (double)snap[(size_t)m * snap_stride + i] - thg;
                sum += delta_m;
            }
            Delta = sum / (double)M;
        }
        /* outer optimizer, Eq. 2 */
        double u_new = mu * (double)u[i] + Delta;
        double G = thg + eta * (Delta + mu * u_new);
        theta_g_out[i] = G;
        u_out[i] = u_new;
        delta_out[i] = Delta;
        sumsq += (long double)Delta * (long double)Delta;
        if (do_merge) {
            for (int m = 0; m < M; ++m) {
                double a = (double)now[(size_t)m * now_stride + i];
                double b = (double)snap[(size_t)m * snap_stride + i];
                now_out[(size_t)m * n + i] =
                    merged_value(a, b, G, lambda, alpha, tau, H, comp_mode, sign_mode);
            }
        }
    }
    return (double)sumsq;
}

/* Delay compensation and merge alone (Algorithm 1), given the new global
 * state G = theta_g_new[i] computed elsewhere. */
void cocodc_oracle_merge_elements(
    long n, int M,
    const float *snap, long snap_stride,
    const float *now, long now_stride,
    const float *theta_g_new,
    double lambda, double alpha, long tau, long H, int comp_mode, int sign_mode,
    double *now_out)
{
    for (long i = 0; i < n; ++i) {
        double G = (double)theta_g_new[i];
        for (int m = 0; m < M; ++m) {
            double a = (double)now[(size_t)m * now_stride + i];
            double b = (double)snap[(size_t)m * snap_stride + i];
            now_out[(size_t)m * n + i] =
                merged_value(a, b, G, lambda, alpha, tau, H, comp_mode, sign_mode);
        }
    }
}

/* What one device contributes to the all-reduce of Section 2.1: the sum over its M local workers
 * of the pseudo-gradients theta^m_{p,t_p} - theta^g_{p,t_p-H}, per element. */
void cocodc_oracle_pseudo_gradient_sum(long n, int M, const float *snap, long snap_stride,
                                       const float *theta_g, double *sum_out)
{
    for (long i = 0; i < n; ++i) {
        double thg = (double)theta_g[i];
        double sum = 0.0;
        for (int m = 0; m < M; ++m)
            sum += (double)snap[(size_t)m * snap_stride + i] - thg;
        sum_out[i] = sum;
    }
}

/* sum of squares of n fp32 values, for the L2 norm of Eq. 10 */
double cocodc_oracle_sumsq(long n, const float *x)
{
    long double s = 0.0L;
    for (long i = 0; i < n; ++i)
        s += (long double)x[i] * (long double)x[i];
    return (double)s;
}
