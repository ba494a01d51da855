"""Oracle of the paper's link model (Section IV-A), test infrastructure only.

Plain Python floats, one function per equation, in the paper's notation.
Pinned by tests/golden/link_hand_example.txt (worked by hand with exact fractions).
"""
import math


def b_id(V):                                   # bits per token id: ceil(log2 |V|)
    return int(math.ceil(math.log2(V))) if V > 1 else 0


def B_hid(d_h, b_h):                           # Eq. 3
    return d_h * b_h


def B_fb(B_hdr_d, b_pos, V):                   # Eq. 4
    return B_hdr_d + b_pos + b_id(V)


def B_u_FH(B_hdr_u, K_r, V, d_h, b_h):         # Eq. 5
    return B_hdr_u + K_r * b_id(V) + K_r * B_hid(d_h, b_h)


def T_comm_FH(B_u, B_feedback, R_u, PER_u, R_d, PER_d, tau_RTT):   # Eq. 6
    return B_u / (R_u * (1 - PER_u)) + B_feedback / (R_d * (1 - PER_d)) + tau_RTT


def B_u1_SH(B_hdr_u, K_r, V):                  # Eq. 7
    return B_hdr_u + K_r * b_id(V)


def B_req(B_hdr_d, m_r, b_pos):                # Eq. 8
    return B_hdr_d + m_r * b_pos


def B_u2_SH(B_hdr_u, m_r, d_h, b_h):           # Eq. 9
    return B_hdr_u + m_r * B_hid(d_h, b_h)


def T_comm_SH(B_u1, B_request, B_u2, B_feedback, R_u, PER_u, R_d, PER_d, tau_RTT):   # Eq. 10
    up = R_u * (1 - PER_u)
    down = R_d * (1 - PER_d)
    return B_u1 / up + B_request / down + B_u2 / up + B_feedback / down + 2 * tau_RTT


def round_cost(*, V, K_r, m_r, d_h, b_h, b_pos, B_hdr_u, B_hdr_d, R_u, R_d, PER_u, PER_d, tau_RTT):
    fb = B_fb(B_hdr_d, b_pos, V)
    out = dict(b_id=b_id(V), B_hid=B_hid(d_h, b_h), B_fb=fb, B_u_FH=B_u_FH(B_hdr_u, K_r, V, d_h, b_h),
               B_u1_SH=B_u1_SH(B_hdr_u, K_r, V), B_req=B_req(B_hdr_d, m_r, b_pos),
               B_u2_SH=B_u2_SH(B_hdr_u, m_r, d_h, b_h))
    out["T_comm_FH"] = T_comm_FH(out["B_u_FH"], fb, R_u, PER_u, R_d, PER_d, tau_RTT)
    out["T_comm_SH"] = T_comm_SH(out["B_u1_SH"], out["B_req"], out["B_u2_SH"], fb, R_u, PER_u, R_d, PER_d, tau_RTT)
    return out
