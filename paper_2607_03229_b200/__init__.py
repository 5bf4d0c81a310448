"""libmpipe_enc for B200: packed variable-length encoder attention and token merge."""
