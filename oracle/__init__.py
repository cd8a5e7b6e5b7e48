"""CPU oracle for path attention over wGraph node KV segments.

TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64 / exact-integer definitions of
what the CUDA path computes, written from the paper's statement of the problem
(Sec. 3: wGraph DAG; Sec. 5: one KV state per operation node, assembled along
the workflow path; Sec. 5 "stateful" caching = one materialised KV per prefix).
It shares no code with the CUDA path and imports nothing from it.  Only the
tests, the smoke check and the benchmark's cpu-baseline leg may import it; the
product path never does.

Pins (tests/test_oracle_*.py): brute-force softmax in pure Python, the
library's scaled_dot_product_attention in fp64, closed forms (identical keys
give the mean of V, constant V, dominant key), request-order / segment-split /
segment-order invariance, the log-sum-exp merge identity, causal-vs-decode
cross check, the paper's five-operation example workflow worked by hand, and
counting / coverage invariants of the tables; for the differential-KV
reconstruction of Sec. 5.1 (residual.py): hand-worked bf16 sums with ties,
identity and cancellation cases, exact rational arithmetic, and a dense
difference built independently of the sparse format.  The paper prints no
numeric value for this path, so every pin is constructed from the mathematics.
"""
