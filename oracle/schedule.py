"""Oracle for the IndexCache layer schedule -- TEST INFRASTRUCTURE ONLY.

Follows the inference loop of Figure 2(b) and the definitions of Sec. 3
"Overview": a pattern string c over {F, S}; an F layer runs its indexer and
overwrites the cached index tensor; an S layer returns the cached tensor of
f(l) = max{ j < l : c_j = F }. The first layer is always F. Layers are 0-based
here (the paper counts from 1).
"""
from __future__ import annotations


def validate(pattern: str) -> None:
    if len(pattern) < 1:
        raise ValueError("empty pattern")
    for ch in pattern:
        if ch not in "FS":
            raise ValueError(f"pattern character {ch!r} is not F or S")
    if pattern[0] != "F":
        raise ValueError("the first layer must be F")


def source_layers(pattern: str) -> list[int]:
    """f(l) for every layer, with f(l) = l on F layers."""
    validate(pattern)
    src = []
    for l, ch in enumerate(pattern):
        if ch == "F":
            src.append(l)
        else:
            j = l - 1
            while pattern[j] != "F":      # max{ j < l : c_j = F }, by direct search
                j -= 1
            src.append(j)
    return src


def run(pattern: str, indexer_of_layer):
    """The loop of Figure 2(b). ``indexer_of_layer(l)`` returns layer l's index
    tensor (Top-k of its indexer scores); it is called on F layers only.
    Returns (per-layer index tensors, number of indexer calls)."""
    validate(pattern)
    out = []
    cache = None
    calls = 0
    for l, ch in enumerate(pattern):
        if ch == "F":
            T = indexer_of_layer(l)
            calls += 1
            cache = T
        else:
            T = cache
        out.append(T)
    return out, calls
