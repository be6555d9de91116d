"""CPU oracle: test infrastructure only (see rgo.cpp).  The product package never imports it."""
