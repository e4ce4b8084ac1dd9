"""Writes closed_forms.txt: values of the one-peak and k-way-tie closed forms of a softmax row,
evaluated with 40-digit arithmetic (mpmath).  It calls neither the oracle nor the CUDA path.

A row with k equal tops of height h over a flat background of V-k zeros has, from the definition
of the softmax confidence c = q(x_0 | x_t) (Section 2, "Sampling in masked dLLMs") and of the
Shannon entropy of that distribution (the token entropy of Section 3.1):
    s      = k + (V - k) e^{-h}
    conf   = 1 / s
    H      = ln s + h (V - k) e^{-h} / s          (nats)
    logp   = -ln s                                 (log-probability of a top token)
    logp0  = -h - ln s                             (log-probability of a background token)

Run:  python tests/golden/make_closed_forms.py > tests/golden/closed_forms.txt
"""
import mpmath as mp

mp.mp.dps = 40
CASES = [(1024, 1, 8), (1024, 1, 12), (126464, 1, 10), (126464, 1, 14), (126464, 1, 16), (152064, 1, 14),
         (126464, 2, 14), (126464, 3, 16), (126464, 4, 20), (1024, 2, 8), (152064, 4, 18), (16, 1, 3), (7, 2, 1.5)]

print("# V k h conf entropy logp_top logp_background   (closed forms; see make_closed_forms.py)")
for V, k, h in CASES:
    h = mp.mpf(h)
    e = mp.e ** (-h)
    s = k + (V - k) * e
    conf = 1 / s
    H = mp.log(s) + h * (V - k) * e / s
    print(V, k, mp.nstr(h, 6), mp.nstr(conf, 17), mp.nstr(H, 17), mp.nstr(-mp.log(s), 17), mp.nstr(-h - mp.log(s), 17))
