"""B200-native paged-KV rollout attention (append, GQA decode, observation-chunk attention)."""
