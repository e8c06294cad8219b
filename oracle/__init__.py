"""Reference implementations used to check the CUDA library.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this
package and this package imports nothing from it.  Contents:

* ``attn``        fp64 decode attention (C, ``attn_oracle.c``) and the
                  log-sum-exp merge rule (numpy)
* ``brute``       pure-Python attention for hand-sized inputs
* ``kv_model``    logical cache content, residency rule, byte accounting
* ``paper_model`` the paper's memory / time formulas
"""
