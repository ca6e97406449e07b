"""CPU oracle for the ABS (adaptive bounded staleness) parameter-server loop.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow, event-driven numpy
restatement of Algorithm 1 of the paper (arXiv 2301.08895) and of the written
numerics contract that the GPU library follows.  It shares no code with the
CUDA path and never imports it; only the test-suite, the smoke check and the
``cpu_baseline`` / ``--impl reference`` legs of the benchmark may import it.
The product library never calls into this package.

Modules
-------
philox   Philox4x32-10 counter-based generator (Salmon et al., SC'11).
timing   job durations in integer ticks (random execution times, Sec. V-A).
models   per-sample losses and minibatch gradients f, grad f (Eq. 1, Eq. 2).
abs_sim  the round loop: arrivals, Eq. 3 update, Eq. 4-6 rules (Algorithm 1).

Parity status: every function here is pinned by a non-GPU test against a
closed form, a brute-force enumeration, a finite-difference check or a
published known-answer vector, except the two items that the paper gives no
numbers for and that are therefore *parity unpinned*: the convergence-rate
bound (Theorem 1 / Corollary 1) and the accuracy curves of Figs. 1-4.
"""
