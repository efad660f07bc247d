"""CPU oracle of the APMSqueeze hot path: test infrastructure, never the product path."""
