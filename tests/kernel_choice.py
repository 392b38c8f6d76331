"""Host-side restatement of which kernel the library picks for a shape (for launch-count expectations)."""


def tokens_stay_in_shared_memory(M, K, from_bf16=False):
    """Weight-streaming kernel: up to 16 tokens with few elements in all (1, 2, 4 or 8 rows kept per n-tile of eight) are
    decoded by the streaming kernel itself, so the product is a single launch.  The limit on rows kept x K is the
    measured break-even of the per-CTA build against the launch it saves: lower when the tokens are first converted
    from BF16 activations."""
    if M > 16:
        return False
    tiles = 1 if M <= 8 else 2
    rows = 1 if M <= 1 else 2 if M <= 2 else 4 if M <= 4 else 8
    elems = tiles * rows * K
    return elems <= (16384 if from_bf16 else 49152) and elems * 2 <= 128 * 1024
