"""CPU oracle (test infrastructure): a plain, slow RNS-CKKS implementation written from
the paper's definitions.  Only tests, the smoke check and the benchmark's CPU-baseline
leg import it; it shares no code with the CUDA package."""
