// Host-side link model of the paper (Section IV-A): payloads and communication
// latency of one round under full-hidden and selective-hidden upload, and the
// protocol rule of Section VII.  Pure arithmetic on the host; no device work.
#include <math.h>
#include <stdint.h>

#include "../../include/wisv.h"

extern "C" {

int wisv_link_cost_round(const wisv_link* l, int32_t V, int32_t K_r, int32_t m_r, wisv_link_cost* out)
{
    if (!l || !out) return WISV_EINVAL;
    if (V < 1 || K_r < 0 || m_r < 0 || m_r > K_r) return WISV_ESHAPE;
    if (!(l->rate_up_bps > 0.0) || !(l->rate_down_bps > 0.0)) return WISV_EINVAL;
    if (!(l->per_up >= 0.0 && l->per_up < 1.0) || !(l->per_down >= 0.0 && l->per_down < 1.0)) return WISV_EINVAL;
    if (l->d_h < 0 || l->b_h < 0 || l->b_pos < 0 || l->hdr_up_bits < 0.0 || l->hdr_down_bits < 0.0 || l->rtt_s < 0.0)
        return WISV_EINVAL;

    int b_id = 0;                                   // ceil(log2 |V|): smallest b with 2^b >= V
    while (b_id < 31 && (1ll << b_id) < (long long)V) ++b_id;
    const double B_hid = (double)l->d_h * (double)l->b_h;                        // Eq. 3
    const double B_fb = l->hdr_down_bits + l->b_pos + b_id;                      // Eq. 4
    const double up = l->rate_up_bps * (1.0 - l->per_up);                        // goodput denominators of Eqs. 6, 10
    const double down = l->rate_down_bps * (1.0 - l->per_down);

    out->b_id = b_id;
    out->B_hid = B_hid;
    out->B_fb = B_fb;
    out->B_u_FH = l->hdr_up_bits + (double)K_r * b_id + (double)K_r * B_hid;     // Eq. 5
    out->B_u1_SH = l->hdr_up_bits + (double)K_r * b_id;                          // Eq. 7
    out->B_req = l->hdr_down_bits + (double)m_r * l->b_pos;                      // Eq. 8
    out->B_u2_SH = l->hdr_up_bits + (double)m_r * B_hid;                         // Eq. 9
    out->T_comm_FH = out->B_u_FH / up + B_fb / down + l->rtt_s;                  // Eq. 6
    out->T_comm_SH = out->B_u1_SH / up + out->B_req / down + out->B_u2_SH / up + B_fb / down + 2.0 * l->rtt_s;  // Eq. 10
    return WISV_OK;
}

int wisv_choose_protocol(double rtt_s)
{
    // Section VII: full-hidden upload when the round-trip time exceeds 10 ms, selective-hidden otherwise
    return rtt_s > 0.010 ? (int)WISV_MODE_FH : (int)WISV_MODE_SH;
}

}  // extern "C"
