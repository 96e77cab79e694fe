"""B200 (sm_100a) library for the partitioned, micro-batch pipelined training step of HyPar-Flow.

Thin ctypes binding over the C ABI declared in include/hpf.h: argument marshalling only.
PyTorch provides device memory and streams; every step of the path runs in the library's kernels.
"""
from .binding import (HpfError, Model, lib, estimate_op_costs, balance_cuts, CONV, BNRELU, ADD, MAXPOOL, HEAD, BN, RELU,
                      OPT_GRAPH, OPT_CONV_PATH, OPT_SINGLE_STREAM, OPT_KEEP_MESSAGES, OPT_FUSE_ADD, OPT_PDL, OPT_WGRAD_PASSES, OPT_FUSE_BN, OPT_CELL_TIMES, OPT_BN_CLUSTER, OPT_CELL_CTAS, OPT_PDL_LATE_FROM, OPT_STAGE_LANES, OPT_WGRAD_DIRECT,
                      conv_fwd, conv_dgrad, conv_wgrad, conv_prepare_weights, conv_scratch_bytes,
                      bnrelu_fwd, bnrelu_bwd, bnrelu_scratch_bytes, bnrelu_status, grad_average_flat, sgd_momentum_flat,
                      bnrelu_fwd_static, static_scratch_bytes)
