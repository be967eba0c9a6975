"""CPU oracle for Hierarchical Speculative Decoding (HSD).

TEST INFRASTRUCTURE ONLY.  This package is a plain, slow restatement of what
the method computes (Algorithm 1, Algorithm 2, the speculative-sampling rule of
Section 2, the latency expression of Theorem 3.2 / Corollary 4.1 and the
hierarchy search of Section 4) plus the sampler / RNG / model-numerics
specification this project fixes where the paper is silent.  Only the test
suite, the smoke check and the CPU-baseline / reference legs of the benchmark
may import it.  It shares no code with the CUDA library and imports nothing
from it; the CUDA library never imports this package.

Pins (what each part is checked against, other than itself):
  philox        known-answer vectors of Philox4x32-10 (Salmon et al. 2011)
  sampling      math.exp / fp64 softmax; exact counting over all 2^24 uniforms;
                closed form 1 - TV(p, q) (Section 2); speculative-sampling lemma
  verify / hsd  exact enumeration against the target's law (Theorem 3.1);
                yield bounds (Section 1); Leviathan et al. closed form for K = 1
  transformer   library routines (torch rms_norm / scaled_dot_product_attention /
                silu) on the same weights; cache == from-scratch
  latency       worked numbers printed in the paper (Table 1, Appendix B grids);
                brute force over (sigma, T)
Parity unpinned: the concrete token ids of a run (fixed only by this project's
sampler specification, nothing external); rows of the paper's worked tables that
its own stated inputs do not reproduce (listed in tests/golden/README.md).
"""
