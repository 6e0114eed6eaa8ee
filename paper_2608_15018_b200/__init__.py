"""B200-native MoE verification layer with reuse-aware expert gating (S2-MoE hot path)."""
