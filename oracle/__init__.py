"""CPU oracle of the Task-KV hot path: test infrastructure, never a product path."""
