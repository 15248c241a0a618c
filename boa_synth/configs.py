"""Workload descriptions for the synthetic inputs.

Each `Workload` describes one seeded synthetic data set shaped like one of the
benchmark configurations: how many points, their dimension and element type,
the cluster mixture they are drawn from, the attribute columns, the proximity
graph's degree and edge mix, the query batch and the selectivity of its range
predicates, and the search parameters (k, L0, Lmax).

This module holds descriptions only.  None of the search method's arithmetic
lives here: both the CPU oracle's tests and the CUDA library's tests import
it, and neither of those two imports the other.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Tuple


@dataclass(frozen=True)
class Workload:
    name: str
    N: int                 # points
    D: int                 # dimension
    vec_dtype: str         # "f32" | "u8"
    vec_kind: str          # "gauss" | "int_latent" | "unit_latent" | "float_latent"
    n_clusters: int
    attrs: Tuple[str, ...]  # attribute column kinds, one per column
    R: int                 # graph out-degree
    graph: str             # "exact_knn" | "mixed"
    Q: int                 # queries in the batch
    sel_kind: str          # "window" | "loguniform" | "mixture"
    sel_lo: float
    sel_hi: float
    k: int
    L0: int
    Lmax: int
    # generator knobs (latent geometry; see generate.py)
    dz: int = 6            # latent dimension of the cluster mixture
    spread: float = 1.0    # std of cluster centres in latent space
    sigma_l: float = 0.6   # within-cluster std in latent space (clusters overlap)
    sigma_n: float = 0.04  # isotropic ambient noise, relative to the latent scale
    # graph knobs for graph == "mixed"
    r_long: int = 6        # multi-scale long edges per node
    long_attr_aware: bool = True  # long edges land on attribute-near points of the far cell
    r_rev: int = 4         # reverse copies of nearest-neighbour edges per node
    r_attr: int = 16       # attribute-window neighbours per node
    attr_fracs: Tuple[float, ...] = (0.1, 0.01)  # fraction of the data inside one attribute window
    t_near: int = 16       # neighbouring cells searched for kNN candidates
    k_cand: int = 64       # nearest candidates the occlusion pruning starts from
    prune_alpha: float = 1.2  # occlusion factor (0 = plain nearest neighbours)

    def scaled(self, N: int, Q: int | None = None, name: str | None = None) -> "Workload":
        """Same recipe at another size; points per cluster kept where possible."""
        per = max(1, self.N // self.n_clusters)
        nc = max(4, min(self.n_clusters, N // per if N // per > 0 else 1))
        return replace(self, N=N, Q=self.Q if Q is None else Q, n_clusters=nc,
                       name=name or f"{self.name}@{N}")

    @property
    def m(self) -> int:
        return len(self.attrs)


# The five benchmark configurations.
C1 = Workload(name="c1_tiny", N=10_000, D=32, vec_dtype="f32", vec_kind="gauss",
              n_clusters=16, attrs=("uniform_int_1000",), R=16, graph="exact_knn",
              Q=100, sel_kind="window", sel_lo=0.10, sel_hi=0.10, k=10, L0=16, Lmax=128)

C2 = Workload(name="c2_int128", N=1_000_000, D=128, vec_dtype="f32", vec_kind="int_latent",
              n_clusters=256, attrs=("uniform_int", "timestamp"), R=32, graph="mixed",
              Q=10_000, sel_kind="loguniform", sel_lo=0.01, sel_hi=0.50, k=10, L0=16, Lmax=512)

C3 = Workload(name="c3_unit96", N=1_000_000, D=96, vec_dtype="f32", vec_kind="unit_latent",
              n_clusters=1024, attrs=("zipf_cat", "uniform_float", "cluster_corr_int"), R=32,
              graph="mixed", Q=10_000, sel_kind="loguniform", sel_lo=0.001, sel_hi=0.01,
              k=10, L0=16, Lmax=512, attr_fracs=(0.01, 0.001))

C4 = Workload(name="c4_u8_10m", N=10_000_000, D=128, vec_dtype="u8", vec_kind="int_latent",
              n_clusters=4096, attrs=("uniform_int", "uniform_int"), R=64, graph="mixed",
              Q=10_000, sel_kind="loguniform", sel_lo=0.005, sel_hi=0.50, k=10, L0=32, Lmax=512,
              r_long=8, r_attr=32, r_rev=8)

C5 = Workload(name="c5_f960", N=1_000_000, D=960, vec_dtype="f32", vec_kind="float_latent",
              n_clusters=512, attrs=("uniform_int", "uniform_float", "zipf_cat", "zipf_cat"),
              R=32, graph="mixed", Q=100_000, sel_kind="mixture", sel_lo=0.001, sel_hi=0.80,
              k=10, L0=16, Lmax=512)

# c1 with a connected graph: the config's literal exact 16-NN graph over 16 well separated
# clusters reaches 5.7 % of the nodes from the entry point, so recall is measured on this
# variant (4 pruned neighbours, 1 reverse, 8 attribute-window, 3 long edges).
C1B = replace(C1, name="c1b_tiny_connected", graph="mixed", t_near=16, r_attr=8, r_long=3, r_rev=1,
              attr_fracs=(0.1,))

ALL = {"c1": C1, "c1b": C1B, "c2": C2, "c3": C3, "c4": C4, "c5": C5}
