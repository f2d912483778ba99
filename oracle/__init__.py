"""CPU oracle (test infrastructure; see xrl_oracle.cpp).  Never imported by the product package."""
