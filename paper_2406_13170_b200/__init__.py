"""B200 (sm_100a) Amphista speculative-decoding step: ctypes binding of libamph.so."""
from .binding import (  # noqa: F401
    AmphError,
    Amphista,
    amph_config,
    amph_tensor,
    amph_tree,
    lib,
    library_path,
    make_config,
    make_tree,
    project,
    project_noalloc,
)
