"""B200-native block-punched CONV / block-based GEMM library (thin Python binding over a C ABI)."""
