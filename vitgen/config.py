"""Model shape description and the named presets used by tests and benchmarks."""
from dataclasses import dataclass, replace


@dataclass(frozen=True)
class ViTConfig:
    image_size: int = 224
    patch_size: int = 16
    channels: int = 3
    hidden: int = 768
    layers: int = 12
    heads: int = 12
    mlp_dim: int = 3072
    num_classes: int = 1000
    ln_eps: float = 1e-6
    extra_tokens: int = 0             # 1 = a distillation token after the class token (the compressed-model family)

    @property
    def grid(self) -> int:            # patches per image side
        return self.image_size // self.patch_size

    @property
    def n_patches(self) -> int:
        return self.grid * self.grid

    @property
    def tokens(self) -> int:          # class token (+ distillation token) + patches
        return self.n_patches + 1 + self.extra_tokens

    @property
    def first_patch_token(self) -> int:
        return 1 + self.extra_tokens

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    @property
    def patch_k(self) -> int:         # length of one flattened patch
        return self.channels * self.patch_size * self.patch_size

    def with_(self, **kw) -> "ViTConfig":
        return replace(self, **kw)


PRESETS = {
    "tiny16": ViTConfig(patch_size=16, hidden=192, layers=12, heads=3, mlp_dim=768),
    "base16": ViTConfig(patch_size=16, hidden=768, layers=12, heads=12, mlp_dim=3072),
    "large16": ViTConfig(patch_size=16, hidden=1024, layers=24, heads=16, mlp_dim=4096),
    "huge14": ViTConfig(patch_size=14, hidden=1280, layers=32, heads=16, mlp_dim=5120),
    # the shape of the "small" compressed model family (same structure, smaller dimensions)
    "small16": ViTConfig(patch_size=16, hidden=384, layers=12, heads=6, mlp_dim=1536),
    # the compressed (distilled) family of the paper's Section 5.5: tiny / small / base dimensions, a
    # distillation token beside the class token (198 tokens) and a second classifier on it
    "deit_tiny16": ViTConfig(patch_size=16, hidden=192, layers=12, heads=3, mlp_dim=768, extra_tokens=1),
    "deit_small16": ViTConfig(patch_size=16, hidden=384, layers=12, heads=6, mlp_dim=1536, extra_tokens=1),
    "deit_base16": ViTConfig(patch_size=16, hidden=768, layers=12, heads=12, mlp_dim=3072, extra_tokens=1),
}


def preset(name: str) -> ViTConfig:
    return PRESETS[name]
