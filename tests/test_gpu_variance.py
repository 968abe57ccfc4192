"""Config 5's variance study on the CUDA path (Sec. 5.1: averaging n_s independent LUQ samples divides
the variance of the weight gradient by n_s and leaves its mean alone; Table 1: Var[SR(x)] = (x-l)(u-x)).
The study itself lives in bench.py (its `variance` block); here its numbers are asserted: the
empirical variances of dW over 256 seed pairs, from the library's quantizer and update GEMM, against
the closed form built from the CPU oracle's bins and codes."""
import pytest
import torch

import bench
from paper_2112_10769_b200 import binding, inputs

pytestmark = pytest.mark.gpu


def test_two_samples_halve_the_variance_and_match_the_closed_form():
    v = bench.variance_study(torch, binding, inputs, 0, rows=4096, block=64, pairs=256)
    assert abs(v["ratio_ns2_over_ns1"] - 0.5) < 0.05, v
    assert abs(v["ns1_over_closed_form"] - 1.0) < 0.10, v
    assert abs(v["ns2_over_closed_form"] - 1.0) < 0.10, v
    assert v["bias_of_block_sum_in_sd"] < 5.0, v
