"""CPU oracle for memory-efficient BPTT (test infrastructure, not a product path).

Everything in this directory is a slow, plain restatement of what the method computes,
written from the paper's equations:

* ``policy``     -- the dynamic programs of Sections 3.1-3.4 (BPTT-HSM / ISM / MSM) and an
                    integer-only simulation of the execution protocol (Algorithm 2 and the
                    prose of Section 3.2) that counts forward operations and memory units.
* ``bruteforce`` -- exhaustive schedule searches over tiny problems that know nothing of
                    the DP tables; they pin ``policy``.
* ``lstm_bptt``  -- standard full-memory BPTT (Section 2.1) of a stacked LSTM with a linear
                    readout and a per-step MSE loss, in float64.

Only the test-suite, the smoke check and the benchmark's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and never receives values from it.
"""
