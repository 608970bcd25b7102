"""CPU checks of the boundary: the shared library loads, exports every symbol the header declares,
and its host-only functions work without a GPU."""
import math
import os
import re

import numpy as np
import pytest
import scipy.special

from paper_2506_06644_b200 import binding as S

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def built():
    from paper_2506_06644_b200 import build
    build.build()
    return S.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "spark.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spark_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(built):
    names = declared_symbols()
    assert sorted(names) == sorted(S.EXPORTS)
    for n in names:
        assert hasattr(built, n), n


def test_status_strings(built):
    seen = {S.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "ok" in seen
    assert S.status_string(99) == "unknown status"


def test_host_quantile_against_library_and_table(built):
    for p in [1e-300, 1e-12, 1e-6, 1e-3, 0.02, 0.08, 0.25, 0.5, 0.75, 0.999, 82 / 1024, 737 / 9216, 256 / 32768]:
        z = S.spark_normal_upper_quantile(p)
        assert abs(z + scipy.special.ndtri(p)) <= 1e-12 * max(1.0, abs(z)), p
    assert abs(S.spark_normal_upper_quantile(0.025) - 1.959963984540) < 1e-11
    assert abs(S.spark_normal_upper_quantile(0.5)) < 1e-15
    for bad in (0.0, 1.0, -0.1, 2.0, float("nan")):
        assert math.isnan(S.spark_normal_upper_quantile(bad))


def test_workspace_bytes_grows_with_the_problem(built):
    a = S.spark_workspace_bytes(1, 9216, 4096, 8, 256, 2304)
    b = S.spark_workspace_bytes(8, 9216, 32768, 8, 256, 2304)
    assert 0 < a < b
    assert b >= 8 * 8 * 32768 * 4                     # room for every predictor score


def test_binding_refuses_to_run_without_a_gpu(built):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(RuntimeError):
        S.SparkContext(0)
