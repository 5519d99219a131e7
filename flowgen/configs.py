"""The five named workload shapes (sizes only; no arithmetic of the method).

Symbols: n flows, N fast-context packets, F statistical features, T trees of
depth d, C classes, P slow-context packets, H header bytes kept per packet.
Seeds: data 1000+c, model 2000+c, validation 3000+c for config number c.
"""
from dataclasses import dataclass, field
from typing import Tuple


@dataclass(frozen=True)
class Config:
    c: int                      # config number 1..5
    name: str
    n: int                      # flows per batch
    N: int                      # packets seen by the fast model
    F: int                      # statistical features (8 per group)
    kind: str                   # "rf" | "gbdt"
    T: int
    depth: int
    C: int                      # classes of the fast model
    P: int                      # packets seen by the slow model
    H: int                      # header bytes per packet in the wide planes
    slow: str                   # "mlp" | "cnn"
    slow_dtype: str             # "f32" | "bf16"
    dims: Tuple[int, ...]       # MLP layer widths, or () for the CNN
    q_percent: int              # Alg. 1 quantile (percent) used for tau; 0 = fixed rule
    n_val: int = 65536          # validation flows for threshold calibration
    cnn: Tuple[int, ...] = ()   # (L, Cin, C1, C2, k, n_cls)
    gbdt_sigma: float = 0.1

    @property
    def seed_data(self) -> int:
        return 1000 + self.c

    @property
    def seed_model(self) -> int:
        return 2000 + self.c

    @property
    def seed_val(self) -> int:
        return 3000 + self.c

    @property
    def D(self) -> int:
        return self.P * 16 if self.slow == "mlp" else self.P * 8

    @property
    def n_slow_classes(self) -> int:
        return self.dims[-1] if self.slow == "mlp" else self.cnn[5]


CONFIGS = {
    1: Config(1, "c1_tiny", 4096, 8, 24, "rf", 16, 8, 4, 64, 13, "mlp", "f32",
              (1024, 256, 256, 4), 75, n_val=4096),
    2: Config(2, "c2_rf100_mlp2048", 1_000_000, 16, 48, "rf", 100, 12, 8, 128, 13, "mlp", "bf16",
              (2048, 1024, 1024, 1024, 8), 76),
    3: Config(3, "c3_gbdt500_mlp1024", 4_000_000, 8, 32, "gbdt", 500, 6, 2, 64, 13, "mlp", "bf16",
              (1024, 512, 512, 2), 0),
    4: Config(4, "c4_rf64_cnn", 1_000_000, 32, 64, "rf", 64, 10, 16, 128, 5, "cnn", "bf16",
              (), 76, cnn=(128, 8, 64, 128, 5, 16)),
    # streaming: the config-2 forest on 8 packets, the config-2 MLP on 64 packets zero-padded to 128
    5: Config(5, "c5_stream", 10_000_000, 8, 48, "rf", 100, 12, 8, 64, 13, "mlp", "bf16",
              (2048, 1024, 1024, 1024, 8), 76),
}


def get_config(c: int) -> Config:
    return CONFIGS[int(c)]
