"""Writes schedule_budgets.txt: the kept-context counts of the three geometric
workload schedules, from the closed form in 50-digit decimal arithmetic
(gamma = (r_end / r_start) ** (1 / (layers - 1)); ratio_l = max(r_end,
r_start * gamma ** l); k_l = min(c_l, floor(ratio_l * c_0))). It calls neither
the oracle nor the library: the file pins the oracle's budget arithmetic.

    python tests/golden/make_schedule_budgets.py
"""
import os
from decimal import Decimal, getcontext, ROUND_FLOOR

getcontext().prec = 50
ROWS = [("7b", 32, 2048, 256, "1.0", "0.3"), ("13b", 40, 4096, 512, "1.0", "0.25"), ("70b", 80, 8192, 1024, "1.0", "0.2")]
HEAD = """# Kept context keys k_l fixed by the workload definitions (integer identities of
# k_l = floor(ratio_l * c_0), geometric ratio clamped at its end value), not by the paper.
# name layers prompt_len recent_len r_start r_end : first six k_l ... last three k_l
"""


def budgets(layers, N, L, r0, r1):
    r0, r1 = Decimal(r0), Decimal(r1)
    gamma = (r1 / r0).ln() / (layers - 1)
    c0 = N - L
    ks, c = [], c0
    for l in range(layers):
        ratio = max(r1, r0 * (gamma * l).exp())
        k = min(c, int((ratio * c0).to_integral_value(rounding=ROUND_FLOOR)))
        ks.append(k)
        c = k
    return ks


if __name__ == "__main__":
    out = HEAD
    for name, layers, N, L, r0, r1 in ROWS:
        ks = budgets(layers, N, L, r0, r1)
        out += f"{name} {layers} {N} {L} {r0} {r1} : {' '.join(map(str, ks[:6]))} ... {' '.join(map(str, ks[-3:]))}\n"
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "schedule_budgets.txt"), "w") as f:
        f.write(out)
