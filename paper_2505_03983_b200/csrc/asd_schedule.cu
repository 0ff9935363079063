// DDPM front end: turns a DDPM noise schedule (alpha-bar per level) and the network's prediction type
// into the inputs of the library's chain (Eq. 7): time grid, per-step variances and the per-step
// scalars c_in / c_skip / c_out that wrap the network into the drift g.  Host arithmetic only (fp64).
//
// Two mappings:
//  * stochastic localization (Theorem 1, with x_t = sqrt(ab) x0 + sqrt(1 - ab) eps):
//        t = ab / (1 - ab),   y = sqrt(t (1 + t)) x_t,   sigma^2 = eta   (Theorem 2);
//    the drift is the posterior mean E[x0 | x_t].
//  * ancestral (the remark after Algorithm 1): the DDPM ancestral step
//        x_{i+1} = a_i x_i + b_i E[x0 | x_i] + s_i xi
//    is the same chain in the variable y_i = x_i / A_i, A_i = a_0 ... a_{i-1}:
//        y_{i+1} = y_i + (b_i / A_{i+1}) E[x0 | x_i] + (s_i / A_{i+1}) xi,
//    i.e. Eq. 7 with eta_i = b_i / A_{i+1} and sigma_{i+1} = s_i / A_{i+1}.
// In both, x_i = x_scale[i] y_i, the network sees c_in[i] y = x_i, and
//        E[x0 | x] = k_x x + k_n net(x):   x0-prediction (0, 1),  eps-prediction (1/sqrt(ab), -sqrt((1-ab)/ab)),
//                                          v-prediction (sqrt(ab), -sqrt(1-ab)),
// so c_skip = k_x x_scale and c_out = k_n.
#include <math.h>

#include "asd.h"

extern "C" asd_status asd_ddpm_schedule(int32_t K, const double* alpha_bar, int32_t pred, int32_t map,
                                        int32_t large_variance, double* t_out, double* sigma2_out, float* c_in,
                                        float* c_skip, float* c_out, double* x_scale) {
  if (K < 1 || !alpha_bar || !t_out || !sigma2_out || !c_in || !c_skip || !c_out || !x_scale) return ASD_ERR_INVALID_ARG;
  if (pred < ASD_PRED_X0 || pred > ASD_PRED_V || (map != ASD_MAP_SL && map != ASD_MAP_ANCESTRAL))
    return ASD_ERR_INVALID_ARG;
  for (int i = 0; i <= K; ++i) {
    if (!(alpha_bar[i] > 0.0 && alpha_bar[i] < 1.0)) return ASD_ERR_INVALID_ARG;
    if (i > 0 && !(alpha_bar[i] > alpha_bar[i - 1])) return ASD_ERR_INVALID_ARG;  // noise must decrease
  }
  if (map == ASD_MAP_SL) {
    for (int i = 0; i <= K; ++i) {
      const double t = alpha_bar[i] / (1.0 - alpha_bar[i]);
      t_out[i] = t;
      x_scale[i] = 1.0 / sqrt(t * (1.0 + t));
    }
    for (int i = 0; i < K; ++i) sigma2_out[i] = t_out[i + 1] - t_out[i];
  } else {
    double A = 1.0;  // A_i
    t_out[0] = 0.0;
    x_scale[0] = 1.0;
    for (int i = 0; i < K; ++i) {
      const double ab_s = alpha_bar[i], ab_r = alpha_bar[i + 1];  // from the noisier level s to level r
      const double alpha = ab_s / ab_r, beta = 1.0 - alpha;
      const double a = sqrt(alpha) * (1.0 - ab_r) / (1.0 - ab_s);
      const double b = sqrt(ab_r) * beta / (1.0 - ab_s);
      const double s2 = large_variance ? beta : beta * (1.0 - ab_r) / (1.0 - ab_s);
      const double A_next = A * a;
      t_out[i + 1] = t_out[i] + b / A_next;
      sigma2_out[i] = s2 / (A_next * A_next);
      x_scale[i + 1] = A_next;
      A = A_next;
    }
  }
  for (int i = 0; i < K; ++i) {
    const double ab = alpha_bar[i];
    double kx = 0.0, kn = 1.0;
    if (pred == ASD_PRED_EPS) {
      kx = 1.0 / sqrt(ab);
      kn = -sqrt((1.0 - ab) / ab);
    } else if (pred == ASD_PRED_V) {
      kx = sqrt(ab);
      kn = -sqrt(1.0 - ab);
    }
    c_in[i] = (float)x_scale[i];
    c_skip[i] = (float)(kx * x_scale[i]);
    c_out[i] = (float)kn;
  }
  return ASD_OK;
}
