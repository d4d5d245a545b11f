"""B200 (sm_100a) implementation of the integer-arithmetic-only convolution layer.

``binding`` exposes the C-ABI library (``libiconv_b200.so``) one to one; ``network``
sequences those calls over a network description.  There is no CPU fallback: importing
``binding`` raises if the compiled library is missing.
"""
