"""CPU oracle (test infrastructure): see pe_oracle.cpp.  Product code never imports this."""
