"""B200-native tensor-core-unit scan: Python binding over the C-ABI library."""
