"""CPU oracle for the Cassandra self-speculative decode step.

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow restatement of what the
paper's method computes, written from the paper's text with numpy (fp64 for
floating point).  It shares no code, tables or helpers with the CUDA library and
is imported only by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The product path never routes through it.

Pins (tests that tie the oracle to the paper / to mathematics, not to itself):
  * printed unary codes 1, 01, 001 and the "ends in 1" rule        (Sec. 4.2)
  * encode->decode round trips keep exactly the kept bits           (Sec. 4.1/4.2)
  * kept counts and the pruning order                               (Sec. 4.2)
  * chunked decoder (Algorithm 1) == sequential decoder             (Sec. 5.1)
  * brute force on tiny tensors
  * size closed form  1 + (1-p)(8 - t + e_bar)  bits per element    (Eq. 2, Sec. 4.2)
  * speculation + verification bits < 16 per element                (Sec. 7.2)
  * Shannon entropy <= mean unary length                            (Sec. 4.2)
  * p = 0, t = 0 degenerates to the bf16 model (all drafts accepted)
  * greedy speculative stream == plain greedy stream for any draft  (Sec. 2.2)
  * greedy acceptance == Eq. 1 with p/q in {0, 1}
  * draft GEMV / attention on decoded operands == library matmul / softmax
  * attention == the library's scaled-dot-product attention, a brute-force
    double loop, and its one-key / equal-keys special cases          (Sec. 2.1)
  * RMSNorm on a hand-computed vector; SwiGLU against its closed form
  * a whole decoder layer == an independent restatement with library ops
  * sampling acceptance: emitted token distributed as the target's
    (chi-square), acceptance probability sum(min(p, q)), Eq. 1 by brute
    force, one-hot distributions reduce to the greedy rule           (Eq. 1)
  * KV records: entry words, raw-exponent escape, per-slice decode
    round trips; Cassandra-2 KV values against the MX definition     (Sec. 4.1-4.3)
  * design objective on hand-computed points                         (Eq. 2)

Parity unpinned (this build's own readings, fixed only by agreement between the
oracle and the CUDA path): the physical superblock layout, the per-row pruning
group and tie-breaks, codebook scope and tie order, the KV codebook freeze
point, the handling of in-flight draft KV entries, and the list of bf16
rounding points in the model forward pass.
"""
