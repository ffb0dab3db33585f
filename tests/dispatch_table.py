"""Which forced kernel must take which parity case, and which it must decline.

The forced-path parity tests run every (case, path) pair.  A pair listed in a TAKES set must run and
match the oracle; a pair not listed must come back as NPAS_ERR_UNSUPPORTED from both the kernel query
and the compute call.  Nothing is skipped at run time: a kernel whose envelope shrinks (or grows)
fails here until the table is edited on purpose.  ``tests/test_dispatch_cpu.py`` checks the same table
without a GPU through the host-only kernel queries.
"""

# block-punched convolution, bf16, bias + residual + ReLU (3x3, stride 1, pad 1 unless stated)
CONV_CASES = [
    dict(N=2, H=14, W=14, C=64, K=64, Mb=16, Nb=8, keep=3),                      # 0 two ragged row tiles per image
    dict(N=1, H=28, W=28, C=64, K=96, Mb=16, Nb=16, keep=3),                     # 1
    dict(N=2, H=7, W=7, C=128, K=64, Mb=32, Nb=32, keep=5),                      # 2
    dict(N=1, H=14, W=14, C=72, K=48, Mb=16, Nb=8, keep=lambda fb, cb: (fb * 4 + cb) % 10),   # 3 odd pair counts, empty blocks, C % 16 != 0
    dict(N=1, H=10, W=20, C=32, K=32, Mb=16, Nb=8, keep=9),                      # 4 dense blocks
    dict(N=1, H=12, W=12, C=64, K=64, Mb=64, Nb=64, keep=2),                     # 5
    dict(N=2, H=9, W=9, C=32, K=32, Mb=16, Nb=8, keep=1, R=1, S=1, pad=0),       # 6 1x1 layer
    dict(N=1, H=13, W=13, C=16, K=32, Mb=16, Nb=8, keep=7, R=5, S=5, pad=2),     # 7 5x5 punched kernels (25 taps)
    dict(N=1, H=56, W=56, C=16, K=16, Mb=16, Nb=16, keep=4),                     # 8
    dict(N=1, H=6, W=126, C=8, K=16, Mb=16, Nb=8, keep=3),                       # 9 widest image the tile takes, C = 8
    dict(N=1, H=6, W=126, C=16, K=16, Mb=16, Nb=8, keep=3),                      # 10
    dict(N=2, H=14, W=14, C=160, K=256, Mb=16, Nb=8, keep=lambda fb, cb: (fb + cb) % 4),   # 11 partial last stage
    dict(N=1, H=28, W=28, C=96, K=64, Mb=32, Nb=32, keep=3),                     # 12
    dict(N=3, H=7, W=7, C=64, K=512, Mb=16, Nb=16, keep=9),                      # 13
    dict(N=2, H=28, W=28, C=64, K=64, Mb=16, Nb=8, keep=3, stride=2),            # 14 strided: even H, two tiles
    dict(N=2, H=15, W=13, C=32, K=32, Mb=16, Nb=16, keep=4, stride=2),           # 15 strided: odd H and W
]
_ALL = set(range(len(CONV_CASES)))
CONV_TAKES = {
    1: _ALL,                              # CUDA cores: everything
    3: _ALL - {14, 15},                   # shared-memory operands: stride 1 only
    6: _ALL - {3, 7, 9},                  # dense operand image: C % 16 == 0, at most 16 taps
    7: {0, 2, 5, 13, 14},                 # CTA pairs: C % 64 == 0 and K % 64 == 0
    8: {1, 2, 5, 8, 12, 13},              # kept pairs only: stride 1, Mb and Nb multiples of 16
}
# the kernel the automatic choice must pick for each case
CONV_AUTO = {i: 6 for i in _ALL}
CONV_AUTO.update({3: 3, 7: 3, 9: 3, 14: 7})     # 14: the strided 3x3 geometry the pair kernel computes by phases

# block-based GEMM, bf16, bias + ReLU
LINEAR_CASES = [
    dict(M=300, I=256, O=256, Bo=64, Bi=64, keep_rows=16, keep_cols=16),           # 0 ragged last row tile
    dict(M=300, I=704, O=320, Bo=64, Bi=64, keep_rows=9, keep_cols=21),            # 1 11 column blocks, 5 row blocks
    dict(M=128, I=128, O=512, Bo=64, Bi=64, keep_rows=32, keep_cols=32),           # 2
    dict(M=77, I=192, O=128, Bo=64, Bi=64, keep_rows=lambda a, b: (a * 29 + b * 13) % 65,
         keep_cols=lambda a, b: (a * 7 + b * 23) % 65),                             # 3 empty, odd and full blocks
    dict(M=200, I=64, O=96, Bo=32, Bi=32, keep_rows=7, keep_cols=11),              # 4
    dict(M=64, I=128, O=64, Bo=16, Bi=64, keep_rows=16, keep_cols=64),             # 5 nothing pruned
    dict(M=300, I=192, O=256, Bo=64, Bi=64, keep_rows=32, keep_cols=32),           # 6 (the residual case)
]
_LALL = set(range(len(LINEAR_CASES)))
LINEAR_TAKES = {
    1: _LALL,
    3: _LALL,                             # gathered kept columns
    5: _LALL,                             # masked dense image by TMA
    6: {0, 2, 3, 6},                      # CTA pairs: O a multiple of 128
}
LINEAR_AUTO = {0: 6, 1: 5, 2: 5, 3: 5, 4: 5, 5: 5, 6: 5}

UNSUPPORTED = 8    # NPAS_ERR_UNSUPPORTED
