"""CPU oracle for the paged-KV suspend / resume / expire path.

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline leg; never by the product package.
"""
from .orc import (  # noqa: F401
    OrcPool, OrcStats, build, bytes_per_token, gather, image_offset, pool_offset, scatter,
    OK, RESIDENT, RECOMPUTE, HOST_FULL, HBM_FULL,
    ERR_INVALID_ARG, ERR_UNKNOWN_REQUEST, ERR_BAD_STATE, ERR_GEOMETRY, ERR_NOMEM,
    ACTIVE, RETAINED, HOST, EXPIRED, LAYER_MAJOR, BLOCK_MAJOR,
)
