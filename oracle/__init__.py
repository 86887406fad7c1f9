"""CPU oracle: plain, slow reference implementations used only to check the CUDA library.

TEST INFRASTRUCTURE.  Nothing under this package is part of the product: only the tests, the
smoke check and the benchmark's CPU-baseline leg import it, and it imports nothing from the
CUDA package.  See the headers of `contract_oracle.c`, `contract.py` and `csf.py` for what each
function computes and which passage of the paper defines it.
"""
