"""Seeded synthetic workloads shared by the oracle's tests and the CUDA library's tests."""
from .configs import ALL, C1, C2, C3, C4, C5, Workload
from .generate import (ATTR_F32, ATTR_I32, SENTINEL, clean_rows, exact_knn_graph,
                       make_workload, reachable_fraction)

__all__ = ["ALL", "C1", "C2", "C3", "C4", "C5", "Workload", "ATTR_F32", "ATTR_I32", "SENTINEL",
           "clean_rows", "exact_knn_graph", "make_workload", "reachable_fraction"]
