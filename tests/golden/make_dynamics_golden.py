"""Writes cartpole_steps.txt and acrobot_rk4_steps.txt: a few worked transitions of the two textbook
systems, evaluated here in float64 straight from their equations of motion (cart-pole with a uniform
pole, explicit Euler tau = 0.02; the double pendulum "book" Lagrangian, one classical RK4 step of 0.2 s).

Independent of both implementations: imports neither the oracle nor the CUDA library, uses libm in
double precision, no specified polynomials, no fixed operation order.  The fp32 oracle must reproduce
these numbers within 2e-7 (tests/test_oracle_golden.py).

    python tests/golden/make_dynamics_golden.py
"""
import math
import os

HERE = os.path.dirname(os.path.abspath(__file__))


def cartpole(s, act):
    x, xd, th, thd = s
    force = 10.0 if act else -10.0
    g, m_cart, m_pole, half_len = 9.8, 1.0, 0.1, 0.5
    total = m_cart + m_pole
    sn, cs = math.sin(th), math.cos(th)
    temp = (force + m_pole * half_len * thd * thd * sn) / total
    thacc = (g * sn - cs * temp) / (half_len * (4.0 / 3.0 - m_pole * cs * cs / total))
    xacc = temp - m_pole * half_len * thacc * cs / total
    nxt = (x + 0.02 * xd, xd + 0.02 * xacc, th + 0.02 * thd, thd + 0.02 * thacc)
    done = int(abs(nxt[0]) > 2.4 or abs(nxt[2]) > 12.0 * 2.0 * math.pi / 360.0)
    return nxt, done


def acrobot_dsdt(s, torque):
    th1, th2, w1, w2 = s
    m1 = m2 = 1.0
    l1 = 1.0
    lc1 = lc2 = 0.5
    i1 = i2 = 1.0
    g = 9.8
    d1 = m1 * lc1 ** 2 + m2 * (l1 ** 2 + lc2 ** 2 + 2 * l1 * lc2 * math.cos(th2)) + i1 + i2
    d2 = m2 * (lc2 ** 2 + l1 * lc2 * math.cos(th2)) + i2
    phi2 = m2 * lc2 * g * math.cos(th1 + th2 - math.pi / 2)
    phi1 = (-m2 * l1 * lc2 * w2 ** 2 * math.sin(th2) - 2 * m2 * l1 * lc2 * w2 * w1 * math.sin(th2)
            + (m1 * lc1 + m2 * l1) * g * math.cos(th1 - math.pi / 2) + phi2)
    dd2 = (torque + d2 / d1 * phi1 - m2 * l1 * lc2 * w1 ** 2 * math.sin(th2) - phi2) / (m2 * lc2 ** 2 + i2 - d2 ** 2 / d1)
    dd1 = -(d2 * dd2 + phi1) / d1
    return (w1, w2, dd1, dd2)


def acrobot_rk4(s, torque, h=0.2):
    def axpy(a, k, y):
        return tuple(yi + a * ki for yi, ki in zip(y, k))
    k1 = acrobot_dsdt(s, torque)
    k2 = acrobot_dsdt(axpy(h / 2, k1, s), torque)
    k3 = acrobot_dsdt(axpy(h / 2, k2, s), torque)
    k4 = acrobot_dsdt(axpy(h, k3, s), torque)
    return tuple(y + h / 6 * (a + 2 * b + 2 * c + d) for y, a, b, c, d in zip(s, k1, k2, k3, k4))


def main():
    with open(os.path.join(HERE, "cartpole_steps.txt"), "w") as f:
        f.write("# CartPole, one explicit-Euler step (tau = 0.02) of the textbook cart-pole equations, evaluated in float64\n"
                "# by make_dynamics_golden.py (no oracle, no CUDA).  The paper (Section 2.2) gives no equations; the task's\n"
                "# config fixes g = 9.8, m_cart = 1, m_pole = 0.1, half-length 0.5, force +-10, done if |x| > 2.4 or |theta| > 12 deg.\n"
                "# Columns: x xdot theta thetadot action -> x' xdot' theta' thetadot' done\n")
        for s, a in [((0.0, 0.0, 0.0, 0.0), 1), ((0.0, 0.0, 0.0, 0.0), 0), ((0.01, -0.02, 0.03, 0.04), 1), ((1.0, 0.5, -0.1, -1.0), 0),
                     ((2.39, 1.0, 0.2, 0.5), 1), ((-2.39, -1.0, 0.05, 0.1), 0), ((0.3, -0.7, 0.2, 1.0), 1)]:
            n, d = cartpole(s, a)
            f.write(" ".join("%.9g" % v for v in s) + " %d " % a + " ".join("%.12f" % v for v in n) + " %d\n" % d)
    with open(os.path.join(HERE, "acrobot_rk4_steps.txt"), "w") as f:
        f.write("# Acrobot (double pendulum, 'book' Lagrangian: masses 1, lengths 1, centres of mass 0.5, inertias 1, g = 9.8),\n"
                "# derivative and one classical RK4 step of 0.2 s, evaluated in float64 by make_dynamics_golden.py (no oracle,\n"
                "# no CUDA).  States stay small enough that the angle wrap and the velocity clip are inactive.\n"
                "# Columns: theta1 theta2 omega1 omega2 torque -> acc1 acc2 | theta1' theta2' omega1' omega2'\n")
        for s, a in [((0.0, 0.0, 0.0, 0.0), 1.0), ((0.0, 0.0, 0.0, 0.0), 0.0), ((0.1, -0.1, 0.05, -0.05), -1.0), ((1.0, 0.5, -0.3, 0.7), 0.0),
                     ((-0.7, 1.2, 0.4, -1.1), 1.0)]:
            d = acrobot_dsdt(s, a)
            n = acrobot_rk4(s, a)
            f.write(" ".join("%.9g" % v for v in s) + " %g " % a + "%.12f %.12f | " % (d[2], d[3]) + " ".join("%.12f" % v for v in n) + "\n")


if __name__ == "__main__":
    main()
