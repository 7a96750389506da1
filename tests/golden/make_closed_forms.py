"""Writes tests/golden/closed_forms.txt.

Every value is a mathematical closed form evaluated with 40-digit arithmetic (mpmath
only: nothing from the CPU checker or the CUDA library is called), so the checker can
be pinned to numbers it did not produce.  The paper prints no worked numeric example
for these ops; the closed forms are the ones its correctness stages imply (Section 4:
identical-value rows, near-zero variance) together with textbook identities of the ops
(softplus, log V for equal logits, the 3-4-5 row, cos / sin of small integers).

Run:  python tests/golden/make_closed_forms.py
"""
import os

from mpmath import mp, mpf, exp, log, sqrt, cos, sin

mp.dps = 40
HERE = os.path.dirname(os.path.abspath(__file__))


def bf16_round(v):
    """Nearest bf16 (8 significant bits, ties to even) of a positive mpf, as mpf."""
    import math
    f = float(v)
    m, e = math.frexp(f)          # f = m * 2**e, 0.5 <= m < 1
    q = mpf(v) / mpf(2) ** (e - 8)  # in [128, 256)
    lo = int(q)
    frac = q - lo
    if frac > mpf(1) / 2 or (frac == mpf(1) / 2 and lo % 2 == 1):
        lo += 1
    return mpf(lo) * mpf(2) ** (e - 8)


rows = []


def add(name, value, why):
    rows.append((name, mp.nstr(value, 25), why))


# softmax of two logits is the logistic sigmoid of their difference
add("softmax2_1_0_first", 1 / (1 + exp(-1)), "softmax([1,0])[0] = 1/(1+e^-1)")
add("softmax2_1_0_second", 1 / (1 + exp(1)), "softmax([1,0])[1] = 1/(1+e)")
# cross-entropy of two logits is the softplus of the gap
add("xent2_1_0_t0", log(1 + exp(-1)), "xent([1,0], t=0) = log(1+e^-1)")
add("xent2_1_0_t1", log(1 + exp(1)), "xent([1,0], t=1) = log(1+e)")
# all-equal logits: loss = log V
for V in (8, 32000, 50304, 128256, 128257):
    add(f"log_{V}", log(V), f"xent of {V} equal logits = log {V}")
# rmsnorm([3,4], w=1, eps=0) = [3,4]/sqrt(12.5)
add("rmsnorm_3_4_first", 3 / sqrt(mpf(25) / 2), "3/sqrt((9+16)/2)")
add("rmsnorm_3_4_second", 4 / sqrt(mpf(25) / 2), "4/sqrt((9+16)/2)")
# constant row c=2, w=1.5, eps = float32(1e-6)
import struct
eps32 = mpf(struct.unpack("f", struct.pack("f", 1e-6))[0])
add("rmsnorm_const_2_w1p5", mpf(3) / sqrt(4 + eps32), "w*c/sqrt(c^2+eps), c=2, w=1.5, eps=fp32(1e-6)")
# near-zero-variance row: c = bf16(1e-30), w = 1, eps = fp32(1e-6); eps dominates
c_tiny = bf16_round(mpf("1e-30"))
add("bf16_of_1e-30", c_tiny, "nearest bf16 to 1e-30")
add("rmsnorm_const_tiny", c_tiny / sqrt(c_tiny * c_tiny + eps32), "c/sqrt(c^2+eps), c=bf16(1e-30)")
add("bf16_of_65000", bf16_round(mpf(65000)), "nearest bf16 to 65000")
# one dominant logit: gap 20 over V-1 = 7 others -> loss at the hot index = log1p(7 e^-20)
add("xent_hot_gap20_V8", log(1 + 7 * exp(-20)), "log(1 + 7 e^-20)")
add("xent_cold_gap20_V8", 20 + log(1 + 7 * exp(-20)), "20 + log(1 + 7 e^-20)")

# rotary embedding (Table 3 "rotary_emb"): pair 0 turns by the position itself (base^0 = 1);
# with Dh = 4 and base = 10000 pair 1 turns by p * 10000^(-1/2) = p / 100
for p_ in (1, 2, 3, 2047):
    add(f"cos_{p_}", cos(mpf(p_)), f"rope pair 0 at position {p_}: (1,0) -> (cos, sin)")
    add(f"sin_{p_}", sin(mpf(p_)), f"rope pair 0 at position {p_}")
    add(f"cos_{p_}_over_100", cos(mpf(p_) / 100), f"rope Dh=4 base=1e4 pair 1 at position {p_}")
    add(f"sin_{p_}_over_100", sin(mpf(p_) / 100), f"rope Dh=4 base=1e4 pair 1 at position {p_}")
# Dh = 128, base = 10000, pair 32: exponent -64/128 = -1/2 again; pair 16: 10000^(-1/4) = 1/10
add("cos_7_over_10", cos(mpf(7) / 10), "rope Dh=128 pair 16 at position 7: angle 7 * 10000^(-1/4)")
add("sin_7_over_10", sin(mpf(7) / 10), "rope Dh=128 pair 16 at position 7")

with open(os.path.join(HERE, "closed_forms.txt"), "w") as f:
    f.write("# name value  # derivation (closed forms, 40-digit mpmath; see make_closed_forms.py)\n")
    for name, val, why in rows:
        f.write(f"{name} {val}  # {why}\n")
print(f"wrote {len(rows)} values")
