"""Writes closed_forms.txt: values that the method's definitions fix in closed form, evaluated in
exact rational arithmetic (no oracle, no GPU code is involved; rerun to regenerate the file).

Sparsity metric (Sec. 3.3, the ratio of attention mass on visual tokens older than the newest w to the
mass on all visual tokens, averaged over image steps t = 1..N):
  uniform attention (all logits equal): step t contributes (t - w) / t for t > w and 0 otherwise, so
      s = [(N - w) - w (H_N - H_w)] / N        with H_n the n-th harmonic number;
  all visual mass on image token 0: step t contributes 1 for t > w, so s = (N - w) / N.
Accumulated attention score (Algorithm 1, running sum of post-softmax attention) under uniform attention
with a prompt of L tokens, observed steps t = n0 - n_obs + 1 .. n0: token j gets 1 / (L + t) from every
observed step t > j.
"""
import os
from fractions import Fraction


def H(n):
    return sum(Fraction(1, k) for k in range(1, n + 1))


def main():
    lines = ["# kind args... value   (see make_closed_forms.py for the formulas; Sec. 3.3 and Algorithm 1)"]
    for N, w in ((576, 32), (64, 16), (4096, 256), (40, 7)):
        s_uniform = (Fraction(N - w) - w * (H(N) - H(w))) / N
        lines.append(f"sparsity_uniform {N} {w} {float(s_uniform):.17g}")
        lines.append(f"sparsity_token0 {N} {w} {float(Fraction(N - w, N)):.17g}")
    for L, n0, n_obs, j in ((64, 288, 288, 0), (64, 288, 288, 100), (64, 288, 288, 287), (64, 288, 24, 0),
                            (64, 288, 24, 280), (5, 17, 6, 3)):
        first = max(j + 1, n0 - n_obs + 1)
        v = sum(Fraction(1, L + t) for t in range(first, n0 + 1))
        lines.append(f"score_uniform {L} {n0} {n_obs} {j} {float(v):.17g}")
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "closed_forms.txt"), "w") as f:
        f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
