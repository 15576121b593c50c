"""CPU oracle (test infrastructure, not the product).  See zipmoe_oracle.c and ffn.py."""
