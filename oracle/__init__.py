"""CPU oracle for the compressed LIEC-SGD iteration (Algorithm 1).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg.  The product library never imports this package.
"""
from .liec_oracle import (IDENTITY, SIGN, TOPK, RANDK, randk_compress, build, lib, scale, sign_compress, step,
                          topk_compress, tree_abs_sum, widen_bf16, StepResult, average_step, mean_params, tree_sumsq,
                          philox4x32_10, subset_scores, subset_from_scores, draw_subsets)

__all__ = ["IDENTITY", "SIGN", "TOPK", "RANDK", "randk_compress", "build", "lib", "scale", "sign_compress", "step",
           "topk_compress", "tree_abs_sum", "widen_bf16", "StepResult", "average_step", "mean_params", "tree_sumsq",
           "philox4x32_10", "subset_scores", "subset_from_scores", "draw_subsets"]
