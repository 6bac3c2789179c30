"""libsea: the SEA attention hot path (estimate -> top-k mask -> sparse attention) for B200."""
