"""CPU checker for the AET-SGD hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, sequential restatement of what the method computes, written
from the paper (Algorithm 2 "Setup", Algorithm 3 "AET-SGD Framework", Eq. 1-3,
Section 3.3 "System model", Section 5 and Appendix Table 2) in fp64 NumPy and
Python integers.  It shares no code with the CUDA library and is imported only
by the tests, the smoke check and the benchmark's CPU-baseline leg; the
product path never calls it.

Modules
  rng       counter-based 64-bit generator, sample indices, integer delay draws
  schedule  s_i = a*i + b, round step sizes, the simulated-time event schedule
  models    softmax regression and ReLU-MLP losses / gradients
  sim       the whole run: clients' local-SGD rounds + ordered server updates

Pins (tests marked "not gpu"): the generator against the published SplitMix64
sequence; the schedule against the paper's printed round counts (110 rounds
for K = 60,000 with s_i = 10 i; the ceil(K/s) column of Table 5) and closed
forms; the round step size against values worked by hand from Section 4.1;
gradients against central finite differences; the bf16 rounding points against a
two-sample 2-2-2 network worked scalar by scalar; one client against a
plain SGD loop; d = 0 against synchronous local SGD; the server rule against
w = w_0 - sum(eta * U); a two-client case worked by hand; a convex case
against a brute-force optimum.

Parity unpinned: nothing here reproduces the paper's accuracy, duration or
speed-up tables (they need its data sets, convolutional models and real
threads).
"""
