"""CPU oracle for the DyBit hot path -- test infrastructure, not a product path.

Only tests, the smoke check and the bench's CPU-baseline leg may import this
package.  See ``dybit_oracle.c`` for the arithmetic and ``dybit_oracle.py``
for the numpy-facing wrapper.
"""
