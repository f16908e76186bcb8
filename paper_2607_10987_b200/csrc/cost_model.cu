// Host-only cost model of the state path: T_transfer = |KV| / BW + delta (Sec. 5.4), the scheduling rule
// pi(S) = transfer iff T_transfer < T_prefill (Sec. 4.6; App. C; App. E step 5), and the pack / unpack term the
// paper's model leaves out.  Plain double arithmetic, one rounding per operation, no device involved.
#include <math.h>
#include <stdint.h>

#include "aaf_kv.h"

extern "C" {

int64_t aaf_kv_state_bytes(int32_t n_layers, int32_t n_kv_heads, int32_t head_dim, int32_t elt_bytes, int64_t n_tokens) {
    if (n_layers < 1 || n_kv_heads < 1 || head_dim < 1 || elt_bytes < 1 || n_tokens < 1) return -1;
    long long v = 2;
    const long long f[5] = {n_layers, n_kv_heads, head_dim, elt_bytes, n_tokens};
    for (long long x : f)
        if (__builtin_mul_overflow(v, x, &v)) return -1;
    return v;
}

double aaf_kv_transfer_time(double kv_bytes, double bandwidth_bytes_per_s, double latency_s) {
    if (!(kv_bytes >= 0.0) || !(bandwidth_bytes_per_s > 0.0) || !(latency_s >= 0.0)) return NAN;
    const double wire = kv_bytes / bandwidth_bytes_per_s;
    return wire + latency_s;
}

double aaf_kv_transfer_time_packed(double kv_bytes, double bandwidth_bytes_per_s, double latency_s,
                                   double pack_rate_bytes_per_s) {
    if (!(pack_rate_bytes_per_s > 0.0)) return NAN;
    const double t = aaf_kv_transfer_time(kv_bytes, bandwidth_bytes_per_s, latency_s);
    const double moved = 2.0 * kv_bytes;               // a pack (or unpack) reads and writes every byte once
    const double pack = moved / pack_rate_bytes_per_s;
    double sum = pack + t;
    sum = sum + pack;
    return sum;
}

int aaf_kv_policy(int local_and_compatible, double t_transfer_s, double t_prefill_s) {
    if (local_and_compatible) return AAF_POLICY_REUSE;
    return t_transfer_s < t_prefill_s ? AAF_POLICY_TRANSFER : AAF_POLICY_RECOMPUTE;
}

}  // extern "C"
