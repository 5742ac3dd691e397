"""CPU oracle for blockwise parallel decoding -- TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy restatement of what the decoding path computes,
written from the paper (Sections 2-4 and 6) and independent of the CUDA
library: it has its own blob parser, its own Transformer forward and its own
decode loops.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may import it; the product path never does.

Pins (see tests/test_oracle_*.py): the Transformer stack is checked against
torch.nn.Transformer in float64, the positional signal against closed forms,
the decode loops against the greedy-equivalence guarantee of Section 3, the
invocation counts of Section 4, the worked trace of Section 7.4, the figures'
narratives and brute-force enumeration on tiny vocabularies.

Parity unpinned: absolute logit values of *trained* models (the paper prints
none and no trained weights exist here); only synthetic-weight consistency
can be checked.
"""
