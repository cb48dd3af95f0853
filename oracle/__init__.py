"""Plain CPU oracle of the speculative-decoding hot path (n-gram drafter, decoder forward,
greedy speculative decoding), written from the paper.

TEST INFRASTRUCTURE ONLY.  Only the tests, the smoke check and the benchmark's CPU-baseline
legs may import it; the product path (the CUDA library and its Python binding) never does
and fails loudly when the CUDA library is missing.  Nothing here shares code with the CUDA path.

Parity status of each part is stated in the module headers: everything is pinned by tests
against brute force, closed forms or library routines, except the readings of the mixture
rule that the paper does not spell out (marked "parity unpinned" in ``drafter``).
"""
