"""CPU oracle of the RegTop-k sparsifier: test infrastructure only (see regtopk_oracle.cpp)."""
