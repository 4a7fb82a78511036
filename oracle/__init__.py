"""CPU oracle of the MTAD / MMTAD verification path: test infrastructure, never imported by the product path."""
