"""fp64 CPU oracle of the GRPO scoring path -- test infrastructure, never a fallback."""
