// Host-side pieces around the distillation step (no device work): key-frame striding (Algorithm 2), the
// key-frame schedule the client's loop produces (Algorithm 4), and the throughput / network-traffic bounds of
// Section 4.4 with Section 5.3's rule for choosing MAX_UPDATES.
#include "../../include/shadowtutor.h"

#include <math.h>

extern "C" {

int32_t st_next_stride(int32_t stride, double metric, double threshold, int32_t min_stride, int32_t max_stride)
{
    // two lines through (THRESHOLD, 1): from (0, 0) below the threshold, to (1, 2) above it
    const double ratio = metric < threshold ? metric / threshold : (metric - 2.0 * threshold + 1.0) / (1.0 - threshold);
    double s = floor(ratio * (double)stride);            // whole frames
    if (!(s >= (double)min_stride)) s = (double)min_stride;   // also catches NaN
    if (s > (double)max_stride) s = (double)max_stride;
    return (int32_t)s;
}

st_status st_client_schedule(int64_t n_frames, const double* metrics, int64_t n_metrics, double threshold,
                             int32_t min_stride, int32_t max_stride, int32_t delay, int64_t* key_frames,
                             int64_t capacity, int64_t* n_key_frames)
{
    if (n_frames < 0 || !n_key_frames || min_stride < 1 || max_stride < min_stride || delay < 1 || !(threshold > 0.0 && threshold < 1.0))
        return ST_ERR_INVALID_ARG;
    if ((n_metrics > 0 && !metrics) || (capacity > 0 && !key_frames)) return ST_ERR_INVALID_ARG;
    // Key frame to key frame, no per-frame bookkeeping.  The reply to the key frame at frame f (updated part and
    // metric) is applied min(delay, MIN_STRIDE) frames later: when it has arrived, or when the client stops to
    // wait for it.  The stride recomputed at that moment is at least MIN_STRIDE, so the frames counted since f
    // have not passed it yet, and the next key frame is frame f + NextStride(stride, metric) whatever the delay.
    int64_t n_keys = 0;
    int32_t stride = min_stride;
    st_status status = ST_OK;
    for (int64_t f = 0; f < n_frames; f += stride) {
        if (n_keys >= n_metrics) { status = ST_ERR_INVALID_ARG; break; }          // this key frame has no metric
        if (n_keys < capacity) key_frames[n_keys] = f;
        else status = ST_ERR_BUFFER_TOO_SMALL;                                     // keep counting
        stride = st_next_stride(stride, metrics[n_keys], threshold, min_stride, max_stride);
        ++n_keys;
    }
    *n_key_frames = n_keys;
    return status;
}

static bool latencies_ok(const st_latencies* L)
{
    return L && L->t_si > 0.0 && L->t_sd >= 0.0 && L->t_ti >= 0.0 && L->t_net >= 0.0;
}

st_status st_throughput_bounds(const st_latencies* L, int32_t min_stride, int32_t max_stride, int32_t max_updates,
                               double* fps_lower, double* fps_upper)
{
    if (!latencies_ok(L) || min_stride < 1 || max_stride < min_stride || max_updates < 0) return ST_ERR_INVALID_ARG;
    const double serial = min_stride * L->t_si + L->t_net + L->t_ti;           // no concurrency on the client
    const double overlapped = fmax(min_stride * L->t_si, L->t_net + L->t_ti);  // full concurrency
    if (fps_lower) *fps_lower = min_stride / (serial + max_updates * L->t_sd);
    if (fps_upper) *fps_upper = max_stride / ((max_stride - min_stride) * L->t_si + overlapped);
    return ST_OK;
}

st_status st_traffic_bounds(const st_latencies* L, double s_net, int32_t min_stride, int32_t max_stride,
                            int32_t max_updates, double* per_second_lower, double* per_second_upper)
{
    if (!latencies_ok(L) || min_stride < 1 || max_stride < min_stride || max_updates < 0 || !(s_net >= 0.0)) return ST_ERR_INVALID_ARG;
    if (per_second_lower) *per_second_lower = s_net / (max_stride * L->t_si + max_updates * L->t_sd + L->t_ti + L->t_net);
    if (per_second_upper) *per_second_upper = s_net / fmax(min_stride * L->t_si, L->t_net + L->t_ti);
    return ST_OK;
}

int32_t st_choose_max_updates(const st_latencies* L, int32_t min_stride, int32_t max_stride, double fps_floor)
{
    if (!latencies_ok(L) || min_stride < 1 || max_stride < min_stride) return -1;
    // fps_lower(m) = MIN / (serial + m t_sd) > floor  <=>  m < (MIN / floor - serial) / t_sd ; checked exactly below
    int32_t best = -1;
    for (int32_t m = 0; m <= 1 << 20; ++m) {
        double lo;
        st_throughput_bounds(L, min_stride, max_stride, m, &lo, nullptr);
        if (lo > fps_floor) best = m; else break;
        if (L->t_sd == 0.0) { best = 1 << 20; break; }    // the bound does not depend on m
    }
    return best;
}

}  // extern "C"
