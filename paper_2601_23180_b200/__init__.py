"""B200-native verify pass of TriSpec (ternary speculative decoding with a lightweight proxy
verifier): tree mask, tree-masked GQA attention, LM-head softmax statistics and the
acceptance / escalation scan, as hand-written sm_100a CUDA behind a C-ABI library.

`inputs` draws the seeded synthetic workloads; `binding` wraps the C-ABI entry points
(argument marshalling only) and is imported lazily because it needs the built library."""
