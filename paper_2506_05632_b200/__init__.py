"""B200-native Gumbel-max list sampling: Python binding of libgls (see include/gls.h)."""
