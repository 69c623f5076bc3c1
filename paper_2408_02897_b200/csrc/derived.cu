// Host-side scalars that follow from the device-written records: the forms of Eq. 3 the probe
// reports (mean and max backward error, norm-wise backward error, relative L2 error, SNR) and the
// four tensor statistics of the Experiments section.  Plain host arithmetic on a few doubles; kept
// behind the C ABI so that no caller re-derives the method's scalars on its own.
#include <math.h>

#include "qm_internal.h"

extern "C" {

qm_status qm_metric_scalars(const qm_metric_result* rec, qm_metric_scalars_t* out) {
  if (!rec || !out) return QM_ERR_INVALID_ARG;
  const double n = rec->count > 0 ? (double)rec->count : 1.0;
  const double sd = rec->sum_diff2, sr = rec->sum_ref2, sn = rec->sum_den2;
  out->mean_be = rec->sum_be / n;
  out->max_be = rec->max_be;
  out->normwise_be = sn > 0 ? sqrt(sd / sn) : 0.0;
  out->rel_l2 = sr > 0 ? sqrt(sd / sr) : 0.0;
  out->snr_db = (sd > 0 && sr > 0) ? 10.0 * log10(sr / sd) : INFINITY;
  return QM_OK;
}

qm_status qm_tensor_moments(const qm_tensor_stats_result* rec, qm_tensor_moments_t* out) {
  if (!rec || !out) return QM_ERR_INVALID_ARG;
  out->mean = out->variance = out->skew = out->kurtosis = 0.0;
  if (rec->count == 0) return QM_OK;
  // central moments from the raw power sums, in extended precision: the subtraction of nearly
  // equal terms loses about (mean / sigma)^k digits, and the 64-bit significand of long double
  // gives eleven more bits than the sums themselves carry
  const long double n = (long double)rec->count;
  const long double mu = rec->sum1 / n, r2 = rec->sum2 / n, r3 = rec->sum3 / n, r4 = rec->sum4 / n;
  const long double m2 = r2 - mu * mu;
  const long double m3 = r3 - 3 * mu * r2 + 2 * mu * mu * mu;
  const long double m4 = r4 - 4 * mu * r3 + 6 * mu * mu * r2 - 3 * mu * mu * mu * mu;
  out->mean = (double)mu;
  out->variance = (double)m2;
  if (m2 > 0) {
    out->skew = (double)(m3 / (m2 * sqrtl(m2)));
    out->kurtosis = (double)(m4 / (m2 * m2));
  }
  return QM_OK;
}

}  // extern "C"
